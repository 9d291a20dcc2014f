/*
 * tri_attention.h -- C ABI of the B200 (sm_100a) TriAttention KV-compression round.
 *
 * One round, per (sequence, layer, KV head) "unit" holding N cached keys:
 *   1. score every key with the offset-averaged trigonometric-series estimate plus the
 *      concentration-weighted norm term, once per query head g of the GQA group, z-score
 *      each head's scores over the unit's keys and take the max over g   (Sections 4.1-4.3);
 *   2. keep the B keys with the highest final score                      (Section 4.3);
 *   3. gather the kept K rows, V rows and positions into compacted slots, in slot order
 *      (the eviction of Section 4.3: the cache physically shrinks to B rows).
 *
 * Conventions
 *   - Every function returns a tri_status and never throws, traps or synchronises the device.
 *   - "host" / "device" on a pointer says where the memory must live.  The caller owns every
 *     buffer it passes, including the workspace; the library owns only tri_ctx.
 *   - All launches go to the CUDA stream passed as `stream` (a cudaStream_t cast to void*,
 *     NULL = the legacy default stream) and are asynchronous.  Errors the host can detect
 *     (bad arguments, workspace too small) return before anything is launched.
 *   - Units are indexed u = (layer * S + seq) * n_kv_heads + kv_head.  Per-unit outputs are
 *     dense in u.  head_dim is 128 (64 frequency bands).
 *   - Band layout (tri_model_desc.pair_layout): 0 pairs components (x[2f], x[2f+1]) as the
 *     rotation matrix of Section 2.1 is written; 1 pairs (x[f], x[f+64]).
 */
#ifndef TRI_ATTENTION_H
#define TRI_ATTENTION_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TRI_OK = 0,
    TRI_ERR_INVALID_ARG = 1,   /* NULL where a pointer is required, bad size or stride         */
    TRI_ERR_UNSUPPORTED = 2,   /* head_dim != 128, group_size > 16, page_size % 16 != 0, ...    */
    TRI_ERR_WORKSPACE = 3,     /* ws_bytes < tri_workspace_bytes(...)                           */
    TRI_ERR_CUDA = 4,          /* a CUDA runtime call failed; see tri_last_cuda_error()         */
    TRI_ERR_DEVICE_CHECK = 5,  /* (reported through *device_status, never returned): a page id or
                                  kept index outside its range; such rows are skipped              */
    TRI_ERR_TIMEOUT = 6        /* (reported through *device_status): a bounded wait inside a kernel
                                  ran out; the kernel returned normally, outputs are unspecified    */
} tri_status;

/* Model and method constants.  Host memory; copied by tri_create. */
typedef struct {
    int32_t n_layers;          /* L                                                            */
    int32_t n_kv_heads;        /* H                                                            */
    int32_t group_size;        /* G query heads per KV head (1..16); query head = kv_head*G+g  */
    int32_t head_dim;          /* must be 128                                                  */
    double  rope_theta;        /* RoPE base theta, omega_f = theta^(-2f/d)      (Section 2.1)  */
    int32_t pair_layout;       /* 0 interleaved, 1 half-split                                  */
    int32_t n_offsets;         /* |D|, 1..64                                                   */
    const int64_t *offsets;    /* host [n_offsets]; the future offsets D of Section 4.2
                                  (the paper's set is {1, 2, 4, ..., 2^16}); values >= 0        */
    int32_t norm_variant;      /* weight of |k_f| in the norm term:
                                  0: E|q_f| - |E q_f|   (Section 4.2, default)
                                  1: E|q_f|             (S_norm^(0) of Section 4.1)
                                  2: none (trigonometric term only)                            */
} tri_model_desc;

typedef struct tri_ctx tri_ctx;

/*
 * Builds the per-model context on the current CUDA device: device copies of the calibration
 * statistics of Section 4.1 and the offset-averaged phasors (1/|D|) sum_delta e^{i omega_f delta}.
 *   q_center     host [L][H*G][128] fp32  E[q_f]: pre-RoPE query centre, in the band layout above
 *   q_mean_norm  host [L][H*G][64]  fp32  E|q_f|
 * Allocates device memory and creates the copy stream and events tri_compress_host uses (the only entry
 * point besides tri_destroy and tri_profile_begin that allocates anything).
 */
tri_status tri_create(const tri_model_desc *desc, const float *q_center, const float *q_mean_norm,
                      tri_ctx **out);
tri_status tri_destroy(tri_ctx *ctx);

/*
 * A view of a K/V cache.  All pointers are device pointers owned by the caller.  Strides are in
 * ELEMENTS of the respective array and must be multiples of 8 (16-byte rows); the innermost
 * (head_dim) stride is 1.
 *
 * contiguous (paged == 0):  row(l, s, h, n) at  l*stride_layer + s*stride_seq + h*stride_head + n*stride_tok
 * paged      (paged == 1):  page = page_table[s*max_pages_per_seq + n / page_size],
 *                           row at  l*stride_layer + page*stride_page + h*stride_head + (n % page_size)*stride_slot
 */
typedef struct {
    void *k;                   /* keys: bf16 post-RoPE (k_kind 0), fp32 pre-RoPE (1), bf16 pre-RoPE (2), e4m3 post-RoPE (3) */
    void *v;                   /* values, bf16 (e4m3 with k_kind 3), same strides as k; NULL = no value cache */
    int32_t k_kind;            /* 0: bf16 as cached by the model (post-RoPE) -- the fast path
                                  1: fp32 pre-RoPE vectors, scored in double (a slow reference-style path)
                                  2: bf16 pre-RoPE vectors (the k_f of Section 4.1 as they are), scored in fp32 with
                                     tabulated distance phasors; p_q - p_k must lie in [0, 2^21)
                                  3: 8-bit post-RoPE keys in e4m3 (4 exponent bits, bias 7, 3 mantissa bits, no
                                     infinities), 128 bytes per row, values in the same format.  The paper has no
                                     8-bit cache; a key counts as the value its byte encodes (a positive scale shared
                                     by a unit's keys drops out of the z-score of Section 4.3).  Widened exactly to f16
                                     in registers, then the same contractions on f16 tensor-core MMAs.  Strides are
                                     multiples of 16 elements.  tri_compress_host does not take this format.
                                  1 and 2 need `positions`, or slot = position                                   */
    int32_t paged;
    int64_t stride_layer, stride_seq, stride_head, stride_tok;
    const int32_t *page_table; /* device [S][max_pages_per_seq]                                  */
    int32_t max_pages_per_seq;
    int32_t page_size;         /* multiple of 16                                                 */
    int32_t n_pages;           /* pages in the pool: ids outside [0, n_pages) are reported through
                                  device_status and their rows skipped; 0 = ids are not checked   */
    int64_t stride_page, stride_slot;
    const int32_t *seq_lens;   /* device [S]: keys currently cached per sequence (source views)  */
    int32_t *positions;        /* device [L][S][H][n_max] original RoPE position per slot, or
                                  NULL meaning position == slot index                           */
    int32_t n_max;             /* row capacity per unit (>= every seq_lens[s])                   */
} tri_cache_view;

/* Bytes of device workspace any of the calls below needs for (S sequences, n_max, budget). */
size_t tri_workspace_bytes(const tri_ctx *ctx, int32_t S, int32_t n_max, int32_t budget);

/*
 * Scoring (Sections 4.1-4.3).  For every unit and key n < seq_lens[s]:
 *   raw[g]   = (1/|D|) sum_{delta in D} S_trig^(g)(k, p_q - p_k + delta) + S_norm^(g)(k)
 *   scores   = max_g (raw[g] - mu_g) / sigma_g,  mu_g, sigma_g over the unit's keys (population
 *              standard deviation; a head with sigma_g = 0 contributes 0).
 *   cur_pos  device [S] int64: p_q, the position of the next query of each sequence
 *   scores   device [U][n_max] fp32 (entries >= seq_lens[s] are not written)
 *   raw      device [U][n_max][G] fp32 or NULL: if given, also receives the un-normalised scores
 *   ws       device workspace, 256-byte aligned
 * V is never read.
 */
tri_status tri_score(tri_ctx *ctx, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                     float *scores, float *raw, void *ws, size_t ws_bytes, void *stream);

/*
 * Top-B retention (Section 4.3).  Per unit keeps the `budget` highest scores among the first
 * seq_lens[s] entries; equal scores: the lower slot wins; seq_lens[s] <= budget keeps all.
 *   scores    device [U][n_max] fp32 (finite values)
 *   kept_idx  device [U][budget] int32: kept slots in ascending order (entries >= count untouched)
 *   kept_cnt  device [U] int32: min(budget, seq_lens[s])
 */
tri_status tri_select(tri_ctx *ctx, const float *scores, const int32_t *seq_lens, int32_t S,
                      int32_t n_max, int32_t budget, int32_t *kept_idx, int32_t *kept_cnt,
                      void *ws, size_t ws_bytes, void *stream);

/*
 * Eviction as an order-preserving gather (Section 4.3):  dst row j <- src row kept_idx[j] for K, V
 * and positions, j < kept_cnt[u].  dst may alias src (same k pointer and strides): rows whose source lies
 * inside the destination range [0, kept_cnt) are then moved tile by tile in ascending order by one thread
 * block per unit (a tile is read completely before it is written), the rows behind them by a second,
 * fully parallel launch; rows already in their slot are not touched.  kept_idx must be ascending.
 * dst->seq_lens is ignored; new_seq_lens (device [S], may be NULL) receives kept_cnt of the
 * sequence.  If dst->positions is given it receives the positions of the kept rows.
 */
tri_status tri_compact(tri_ctx *ctx, const tri_cache_view *src, const int32_t *kept_idx,
                       const int32_t *kept_cnt, int32_t S, int32_t budget, const tri_cache_view *dst,
                       int32_t *new_seq_lens, void *stream);

/*
 * The fused round: score, select, compact, in one call (a handful of launches, no host sync).
 * Sequences with seq_lens[s] <= budget are kept whole (Section 4.3 prunes only a cache that has outgrown its
 * budget): their keys are neither scored nor read, so a batch in which only some sequences are due costs
 * only those.
 *   kept_idx, kept_cnt   device outputs as in tri_select, or NULL to use workspace
 *   new_seq_lens         device [S] or NULL: receives min(budget, seq_lens[s]).  It MAY be the same array as
 *                        src->seq_lens (a decode loop that updates its lengths in place): the lengths are
 *                        stored by the last launch of the round only, after every kernel that reads them.
 *   device_status        device int32[1] or NULL; set to TRI_ERR_DEVICE_CHECK if a kernel met a
 *                        page id outside [0, n_pages) -- such rows are skipped, never dereferenced --
 *                        or to TRI_ERR_TIMEOUT if a bounded wait of the scoring kernel ran out
 */
tri_status tri_compress(tri_ctx *ctx, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                        int32_t budget, const tri_cache_view *dst, int32_t *kept_idx,
                        int32_t *kept_cnt, int32_t *new_seq_lens, int32_t *device_status,
                        void *ws, size_t ws_bytes, void *stream);

/*
 * Head-specific budgets (Appendix A lists them as future work; the paper gives no allocation rule, so the budgets
 * are the caller's).  The same calls with one budget per unit:
 *   unit_budgets   device [U] int32; unit u keeps min(unit_budgets[u], budget, seq_lens[s]) rows (negative = 0)
 *   budget         now only the capacity: row stride of kept_idx and upper bound of every unit's budget
 * kept_cnt [U] is the per-unit row count afterwards.  A cache view carries one length per sequence, so new_seq_lens[s]
 * receives the largest count among the sequence's units; rows between a unit's own count and that length are stale,
 * and a later round over such a cache has to be issued per group of units with equal length.
 */
tri_status tri_select_budgets(tri_ctx *ctx, const float *scores, const int32_t *seq_lens, int32_t S,
                              int32_t n_max, int32_t budget, const int32_t *unit_budgets, int32_t *kept_idx,
                              int32_t *kept_cnt, void *stream);
tri_status tri_compress_budgets(tri_ctx *ctx, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                                int32_t budget, const int32_t *unit_budgets, const tri_cache_view *dst,
                                int32_t *kept_idx, int32_t *kept_cnt, int32_t *new_seq_lens,
                                int32_t *device_status, void *ws, size_t ws_bytes, void *stream);

/*
 * The round behind its window trigger (Section 4.3: pruning runs once per window of beta = 128 decoded tokens, and only on
 * a cache that exceeds its budget), decided on the device so that a decode loop -- or a captured CUDA graph -- can issue
 * this call after every step and have it do nothing until a sequence is due.
 *   decoded   device [S] int32, owned by the caller, zero at the start of a sequence: tokens decoded since the
 *             sequence's last window boundary.  The call adds `step` (tokens appended since the previous call); where
 *             the sum reaches `beta` the count starts over and the sequence is due if seq_lens[s] > budget.
 * Due sequences are compressed exactly as by tri_compress.  For the others no key is read and no row moves; their
 * kept_cnt entries are 0, their kept_idx entries untouched and new_seq_lens[s] = seq_lens[s] (the two may be one array).
 * Everything else as in tri_compress; a call in which nothing is due costs the round's launches, whose blocks exit at once.
 */
tri_status tri_compress_windowed(tri_ctx *ctx, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                                 int32_t budget, int32_t *decoded, int32_t step, int32_t beta,
                                 const tri_cache_view *dst, int32_t *kept_idx, int32_t *kept_cnt,
                                 int32_t *new_seq_lens, int32_t *device_status, void *ws, size_t ws_bytes,
                                 void *stream);

/*
 * The fused round for a cache that lives in HOST memory (contiguous views only): copies K of src to the
 * device staging view, runs tri_compress, and copies the compacted rows, positions and counts back, all
 * on `stream`.  V and positions are needed only for the kept rows: if at most half of the rows can be kept
 * (2 * budget <= n_max) and their host arrays are pinned and mapped (cudaHostAlloc / cudaHostRegister), the
 * gather reads those rows directly from host memory and no bulk copy of them is made; otherwise they are
 * staged like K.  The work is pipelined over up to 8 ranges of layers: a range's results travel back on a copy stream owned by the context while the next range is coming
 * in; `stream` waits for that stream at the end, so work enqueued on it after the call sees the host outputs.
 * One context must not run two tri_compress_host calls at once.
 *   src_host / dst_host  views whose k, v, positions, seq_lens pointers are (pinned) host memory
 *   src_dev  / dst_dev   device views of identical shape used as staging (caller-allocated)
 *   cur_pos_host         host [S] int64;  cur_pos_dev device [S] staging
 *   kept_cnt_host        host [U] int32 output
 */
tri_status tri_compress_host(tri_ctx *ctx, const tri_cache_view *src_host, const tri_cache_view *src_dev,
                             int32_t S, const int64_t *cur_pos_host, int64_t *cur_pos_dev, int32_t budget,
                             const tri_cache_view *dst_host, const tri_cache_view *dst_dev,
                             int32_t *kept_cnt_host, int32_t *kept_cnt_dev,
                             void *ws, size_t ws_bytes, void *stream);

/*
 * tri_score without a workspace argument (the paper has no counterpart; this is a packaging variant
 * of tri_score for callers that have nowhere to get scratch memory from at call time).  Examples: an
 * inference server that gave every spare byte of HBM to its KV page pool at start-up, so that a later
 * cudaMalloc fails; a plug-in that is handed raw device pointers by a host application and must keep
 * out of that application's allocator; a latency-critical loop that cannot afford the device-wide
 * synchronisation an allocation may imply.
 *
 * Same arguments, outputs and arithmetic as tri_score, minus ws / ws_bytes.  The phasors, raw scores
 * and partial sums live in one array of TRI_SCORE_STATIC_SCRATCH_BYTES bytes that is compiled into
 * the library as a device global: every GPU on which the library's module gets loaded holds those
 * bytes until the process exits, whether or not this function is ever called.
 *   - The call needs S*1024 bytes of phasors, U*n_max*G*4 bytes of raw scores and 16*G bytes of
 *     partial sums per scoring block (about one block per 1,536 keys), U = n_layers*S*n_kv_heads.
 *     If that exceeds the array the call launches nothing, returns TRI_ERR_WORKSPACE and leaves
 *     both sizes in tri_last_cuda_error().  With G = 4 the array covers about 1.0 M keys per call
 *     (e.g. one layer of 8 KV heads at 128 K keys each).
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, which
 *     may load the module); make that first call during set-up, outside any stream capture.  No call
 *     allocates or frees device memory, and the context must have been created on the current device.
 *   - All calls on a device share the one array and it keeps what the last call left.  Nothing in it
 *     has to start at zero (every word that is read was written earlier in the same call), so it is
 *     never cleared; but two calls whose kernels overlap on the GPU (different streams, or
 *     different host threads on different streams) race on it.  Keep them on one stream or order them
 *     with events.
 */
#define TRI_SCORE_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
/* Bytes of the built-in array a call of tri_score_static with this shape would use (0 for bad arguments). */
size_t tri_score_static_bytes(const tri_ctx *ctx, int32_t S, int32_t n_max);
tri_status tri_score_static(tri_ctx *ctx, const tri_cache_view *src, int32_t S, const int64_t *cur_pos,
                            float *scores, float *raw, void *stream);

/*
 * How tri_compress is issued (the paper has no counterpart; a scheduling choice of this library).
 *   ranges = 1   (default) every kernel of the round on the caller's stream, one launch each.
 *   ranges > 1   the units are cut into that many contiguous ranges (at most 16).  The caller's stream scores range
 *                after range; selection and compaction of a range run on a high-priority stream owned by the context
 *                while the next range is being scored, so the latency-bound selection overlaps the key stream.  The
 *                caller's stream waits for that stream before tri_compress returns control to it: work enqueued on
 *                `stream` afterwards sees the finished round, and a stream capture sees the side stream joined.
 *   ranges = 0   chosen per call: about one range per 32 units, at most 8.
 * Results are bit-identical in every mode.  One context must not run two tri_compress calls concurrently.
 * On B200 the single-stream order measured fastest on every benchmark shape (the selection blocks take shared
 * memory and thread slots from the scoring blocks they overlap), which is why it is the default.
 */
tri_status tri_set_pipeline(tri_ctx *ctx, int32_t ranges);

/*
 * Which kernel scores bf16 keys (the paper has no counterpart; both compute the same Sections 4.1-4.2 scores to
 * fp32 rounding, so results may differ in the last bits between the two, never within one):
 *   0   tcgen05: 128-key tiles, accumulator and magnitude operand in tensor memory (default for group_size > 4)
 *   1   mma.sync: 16-key warp tiles, everything in registers (default for group_size <= 4)
 * Call it before tri_workspace_bytes: the workspace layout depends on the kernel's block size.
 */
tri_status tri_set_score_kernel(tri_ctx *ctx, int32_t which);

/* Number of kernel launches one tri_compress call issues for this shape and mode (for launch accounting). */
int32_t tri_compress_launches(const tri_ctx *ctx, const tri_cache_view *src, int32_t S, const tri_cache_view *dst);

/*
 * Measurement aid (the paper has no counterpart): between tri_profile_begin and tri_profile_end every
 * tri_compress call records a CUDA event before and after each of its launches, on the stream the launch
 * goes to.  tri_profile_read waits for the last call's events and writes the summed durations per kind of
 * kernel in milliseconds to ms[0..4] (host): phasor fold, raw scoring, z-score/max (0 in the fused round,
 * whose selection normalises), top-B select, gather.  In a pipelined round kernels of different kinds overlap,
 * so the five figures may add up to more than the round took.
 * tri_profile_begin creates the events; it is the only one of the three that allocates.
 */
tri_status tri_profile_begin(tri_ctx *ctx);
tri_status tri_profile_read(tri_ctx *ctx, float *ms);
tri_status tri_profile_end(tri_ctx *ctx);

/*
 * Calibration statistics (Section 4.1 takes E[q_f] and E|q_f| from a calibration set; Section 3.3; Appendix B.5).
 * For one layer's query heads, from pre-RoPE query vectors of calibration tokens:
 *   E[q_f]   complex mean per band              -> q_center    [n_heads][128] fp32, in the input's component layout
 *   E|q_f|   mean band magnitude                -> q_mean_norm [n_heads][64]  fp32
 *   R_f = |E[q_f]| / E|q_f|  (mean resultant length, 0 where E|q_f| = 0)  -> mrl [n_heads][64] fp32, may be NULL
 * which are exactly the two arrays tri_create takes.  The statistics are streamed: tri_calib_reset zeroes a
 * running state, tri_calib_accumulate adds T more tokens (call it once per chunk of the calibration set),
 * tri_calib_finalize turns the state into means.  All device pointers; all calls asynchronous on `stream`.
 *   state   device, tri_calib_state_bytes(n_heads) bytes, 8-byte aligned: fp64 sums and the token count
 *   q       device [T][n_heads][128]: bf16 (q_kind 0) or fp32 (q_kind 1); stride_tok / stride_head in elements,
 *           multiples of 4 (q_kind 0: 8-byte rows) resp. 4 (q_kind 1: 16-byte rows); q aligned likewise
 *   ws      device scratch of tri_calib_workspace_bytes(n_heads, T) bytes, 8-byte aligned
 * Sums are formed in a fixed order (no atomics), so equal inputs give equal bits.
 * Rows reach the SMs through the TMA unit when q is 16-byte aligned, both strides are multiples of 16 bytes and
 * T < 2^31 (every contiguous tensor, every fp32 layout accepted here), through plain loads otherwise; the two paths
 * cut the tokens into blocks alike and differ only in speed.  Every wait on a TMA copy is bounded: should one run
 * out, the sums of the pass are set to NaN, so that tri_calib_finalize yields NaN instead of wrong means.
 */
size_t     tri_calib_state_bytes(int32_t n_heads);
size_t     tri_calib_workspace_bytes(int32_t n_heads, int64_t T);
tri_status tri_calib_reset(void *state, int32_t n_heads, void *stream);
tri_status tri_calib_accumulate(const void *q, int32_t q_kind, int64_t T, int32_t n_heads, int64_t stride_tok,
                                int64_t stride_head, int32_t pair_layout, void *state, void *ws, size_t ws_bytes,
                                void *stream);
tri_status tri_calib_finalize(const void *state, int32_t n_heads, int32_t pair_layout, float *q_center,
                              float *q_mean_norm, float *mrl, void *stream);

/*
 * Self-test of the bounded waits the scoring kernels use for their copy-engine and tensor-core barriers (the paper has no
 * counterpart): one warp waits on a barrier that nothing ever completes, once with the spinning wait of the mma.sync
 * kernel and once with the sleeping wait of the tcgen05 kernel; each gives up after a short poll limit.  *device_status
 * (device int32) ends as TRI_ERR_TIMEOUT if both ran out, as TRI_ERR_DEVICE_CHECK if a wait claimed success; the kernels
 * return normally and the context stays usable.
 */
tri_status tri_selftest_bounded_wait(int32_t *device_status, void *stream);

/* Text of the last CUDA error seen by this library on the calling thread ("" if none). */
const char *tri_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TRI_ATTENTION_H */

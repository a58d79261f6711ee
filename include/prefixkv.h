/*
 * prefixkv.h -- C ABI of the B200 (sm_100a) PrefixKV hot-path library.
 *
 * PrefixKV (arXiv 2412.03409) compresses the KV cache of a transformer after
 * prefilling: every prompt key/value vector gets an importance score from the
 * causal attention it receives (Sec. 3.2); each layer's vectors are ranked by
 * that score and their normalised importance is accumulated along the ranking
 * (the "cumulative priority"); one global information-retention ratio p, found
 * by binary search, fixes how long a prefix of each layer's ranking is kept so
 * that the total meets a budget (Sec. 3.3, Eq. 1, Algorithm 1); the kept rows
 * form per-layer caches of unequal length that decoding then attends over
 * (Sec. 3.1, Fig. 2a).
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer unless its comment says "host".  Structs
 *    passed by pointer (pkv_shape, pkv_cache) live on the host.
 *  - The caller owns and allocates every buffer, including workspace; the
 *    library never allocates or frees device memory.
 *  - Every call only enqueues work on `cuda_stream` (a cudaStream_t passed as
 *    void*; NULL = default stream) and returns at once.  The int returned is a
 *    pkv_status from host-side argument validation.  Nothing is synchronised
 *    and no value is read back to the host.
 *  - Conditions found on the device are reported per sample in dev_status[B]
 *    (PKV_DEV_*).  A kernel that finds one still finishes and never touches
 *    memory outside the caller's buffers; the results of that sample are then
 *    unspecified.  prefixkv_search / prefixkv_apply_lengths overwrite
 *    dev_status; later stages only raise it from PKV_DEV_OK.
 *  - Logical tensor shapes use B (batch), L (layers), H (heads), N (prompt
 *    tokens), D (head_dim).  "Segment" = one (sample, layer) pair, index b*L+l.
 *  - Supported: dtype fp32 or bf16; head_dim 64 or 128; N <= 16384;
 *    H*D*sizeof(element) a multiple of 16 bytes.
 */
#ifndef PREFIXKV_H_
#define PREFIXKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PKV_OK = 0,
    PKV_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, bad range, misalignment   */
    PKV_ERR_UNSUPPORTED = 2, /* dtype / head_dim / prompt_len outside the supported set     */
    PKV_ERR_WORKSPACE = 3,   /* workspace missing, misaligned (256 B) or too small          */
    PKV_ERR_CUDA = 4,        /* a CUDA runtime call failed (see prefixkv_last_cuda_error)    */
    PKV_ERR_STATIC_LIMIT = 5 /* shape too large for the built-in scratch of a *_static call */
} pkv_status;

enum { /* per-sample device status word */
    PKV_DEV_OK = 0,
    PKV_DEV_BAD_SCORE = 1,        /* NaN, inf or negative importance                   */
    PKV_DEV_RANGE = 2,            /* fixed-point importance total >= 2^53               */
    PKV_DEV_BUDGET_TOO_SMALL = 3, /* budget < L (each layer keeps at least one row)     */
    PKV_DEV_BAD_LENGTH = 4,       /* a given length outside [1, N]                      */
    PKV_DEV_CAPACITY = 5,         /* rows would pass a segment's or the cache's capacity */
    PKV_DEV_TIMEOUT = 6           /* a bounded wait inside a kernel ran out (reported on sample 0) */
};

typedef enum { PKV_F32 = 0, PKV_BF16 = 1 } pkv_dtype;

typedef struct {
    int32_t batch, layers, heads, head_dim, prompt_len;
    int32_t dtype; /* pkv_dtype */
} pkv_shape;

/* Element strides of a [B, L, H, N, D] tensor; the D stride is 1. */
typedef struct {
    int64_t b, l, h, n;
} pkv_strides;

enum { PKV_WS_SCORE = 0, PKV_WS_SEARCH = 1, PKV_WS_COMPACT = 2, PKV_WS_DECODE = 3 };

/* Bytes of 256-byte-aligned workspace the named call needs for this shape.
 * Returns 0 for an unknown `which` or an unsupported shape. */
size_t prefixkv_workspace_bytes(const pkv_shape *shape, int which);

/* Text of the last CUDA error seen by this library on the calling thread (host). */
const char *prefixkv_last_cuda_error(void);

/*
 * Importance score, Sec. 3.2:
 *   a^{h,m,n} = softmax over keys j <= m of scale_l * <q^{h,m}, k^{h,j}>   (causal)
 *   I[b,l,n]  = (1/H) * sum_h sum_{m >= n} a^{h,m,n}
 * over all N prompt queries.  The printed formula has no scale; scale_l = 1
 * reproduces it.
 *   q, k        [B,L,H,N,D] with the given element strides (D contiguous; every
 *               stride a multiple of 8 elements for bf16 / 4 for fp32 so that
 *               rows start on 16 bytes)
 *   layer_scale [L] fp32
 *   lse         [B,L,H,N] fp32 or NULL: natural-log sum-exp of each query's scaled
 *               causal logits, if the caller's prefill attention kept it; when
 *               NULL the library computes it in a first pass
 *   scores      [B,L,N] fp32, out
 * bf16 inputs use tensor cores with fp32 accumulation; fp32 inputs use fp32 FMA (so do
 * bf16 inputs whose strides no tensor map can describe, e.g. a zero stride).
 * The workspace holds per-head partial sums and work counters: calls that share one must
 * not overlap on the GPU.  The call has no status argument: if a bounded wait inside the
 * tensor-core kernel runs out, every score of the call is written as NaN, which
 * prefixkv_search / prefixkv_apply_lengths report as PKV_DEV_BAD_SCORE.
 */
int prefixkv_score(const pkv_shape *shape, const void *q, pkv_strides qs, const void *k,
                   pkv_strides ks, const float *layer_scale, const float *lse, float *scores,
                   void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Priority sequence, cumulative priority and the binary search for p
 * (Sec. 3.2, Sec. 3.3, Eq. 1, Algorithm 1), per sample.
 *   scores        [B,L,N] fp32, finite and >= 0
 *   budget_rows   [B] int64: total rows the sample may keep over all layers
 *                 (the paper's r*L*N); must be >= L
 *   order         [B,L,N] int32 out: positions by (score descending, position
 *                 ascending) -- the sorted indices s_l^j
 *   cum           [B,L,N] uint64 out: inclusive prefix sums along `order` of
 *                 round-half-even(score * 2^32); cum[..,N-1] is the layer total,
 *                 so P_l^{j/N} = cum[j-1] / cum[N-1]
 *   len           [B,L] int32 out: rows kept per layer (R_l * N), each in [1,N]
 *   p_out         [B] fp64 out: the ratio p the lengths belong to
 *   iters_out     [B] int32 out: midpoints evaluated
 * Length rule: p >= 1 keeps N rows; otherwise theta = ceil(p * total) (one fp64
 * multiply) and len = first 1-based j with cum[j-1] >= theta.
 * Search: if L*N <= budget, p = 1.  Else bisect [0,1]: stop when the interval is
 * <= tol wide, after max_iters midpoints, or when fp64 cannot split it.  With
 * delta = S - budget for a midpoint's total S: a midpoint with
 * -slack_rows <= delta <= slack_over_rows is returned at once (delta = 0 always
 * is); delta < 0 raises the lower end, otherwise the upper end drops.  On a stop
 * the lower end is returned, whose total never exceeds the budget.
 * The two slacks are the threshold on delta of Sec. 3.3 (Tab. "robustness-delta"
 * states it as a fraction of sum R_l; here it is a number of rows, per side).
 * slack_over_rows = 0 keeps sum(len) <= budget.  slack_rows = slack_over_rows is
 * the printed |delta| <= threshold: the configuration may then exceed the budget
 * by up to that many rows and is to be scaled back with prefixkv_rescale before
 * prefixkv_compact.
 */
int prefixkv_search(const pkv_shape *shape, const float *scores, const int64_t *budget_rows,
                    double tol, int32_t max_iters, int64_t slack_rows, int64_t slack_over_rows,
                    int32_t *order, uint64_t *cum, int32_t *len, double *p_out, int32_t *iters_out,
                    int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Variant for a configuration fixed in advance (the offline estimate of
 * Sec. 3.3, last paragraph, or the uniform R_l = r of Sec. 3.2): ranks the rows
 * as above and takes the lengths from the caller.
 *   len_in   [L] (per_sample = 0) or [B,L] (per_sample = 1) int32, each in [1,N];
 *            must not be the same buffer as `len`
 *   cum      may be NULL
 */
int prefixkv_apply_lengths(const pkv_shape *shape, const float *scores, const int32_t *len_in,
                           int32_t per_sample, int32_t *order, uint64_t *cum, int32_t *len,
                           int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Meeting the budget exactly after the search (Sec. 3.3 has the configuration found scaled to
 * the target budget and prints no formula).  Reading: every layer keeps its one mandatory row
 * and the other budget - L rows are split in proportion to len - 1: floor of the quota first,
 * at most N rows per layer, then what is left over one row at a time in the order of the
 * division remainders (largest first, ties to the lower layer), round after round, to the
 * layers that still have room.  The result sums to min(budget, L*N) exactly.  A configuration
 * that already sums to its budget is left unchanged; one below it only grows (each layer keeps
 * a longer prefix of the same priority sequence); one above it -- a search ended by
 * slack_over_rows -- only shrinks, never below one row per layer.
 *   len          [B,L] int32, in/out (from prefixkv_search)
 *   budget_rows  [B] int64
 * Call it between prefixkv_search and prefixkv_compact.
 */
int prefixkv_rescale(const pkv_shape *shape, int32_t *len, const int64_t *budget_rows,
                     int32_t *dev_status, void *cuda_stream);

/*
 * Offline configuration (Sec. 3.3, last paragraph: the lengths found on a few sample prompts
 * are applied to every input; the aggregation is not specified).  Reading: the same
 * apportionment with weight[l] = sum over the B sample prompts of (len[b][l] - 1).
 *   len          [B,L] int32: per-sample lengths of B sample prompts (prefixkv_search)
 *   budget_rows  host value: rows the configuration may keep over all layers
 *   len_out      [L] int32 out: pass it to prefixkv_apply_lengths with per_sample = 0
 *   dev_status   [B]; conditions are reported on sample 0
 */
int prefixkv_estimate_config(const pkv_shape *shape, const int32_t *len, int64_t budget_rows,
                             int32_t *len_out, int32_t *dev_status, void *cuda_stream);

/*
 * Ragged per-layer cache (Fig. 2a).  Rows of segment s occupy
 * [row_offset[s], row_offset[s] + cap[s]) of k and v; the first len[s] are
 * valid.  A row is one token's vectors for all heads: [H][D] elements.
 */
typedef struct {
    void *k;                /* [total_cap_rows][H][D], caller-allocated                  */
    void *v;                /* same                                                      */
    int64_t *row_offset;    /* [B*L + 1] out: exclusive prefix sum of cap                */
    int32_t *len;           /* [B*L] out: valid rows; grows by one per decode step       */
    int32_t *cap;           /* [B*L] out: len after compaction + decode_cap              */
    int64_t total_cap_rows; /* host: rows allocated; must cover sum(len) + B*L*decode_cap */
    int32_t decode_cap;     /* host: rows of head-room per segment for decoding          */
    /* Decode-time pruning (optional; evict_distance = 0 or NULL pointers: the cache only grows). */
    int32_t evict_distance; /* host: d > 0 drops the token generated d steps ago when a layer
                               would exceed its proportion len0 / N of the sequence            */
    int32_t *len0;          /* [B*L] out: rows kept by compaction                              */
    int32_t *gen;           /* [B*L] out: tokens decoded so far                                */
    int32_t *slot_ring;     /* [B*L][evict_distance + 1] out: row of each recent token, -1 once dropped */
} pkv_cache;

/*
 * Compression after prefilling (Sec. 3.1; Sec. 3.2: each layer keeps its R_l
 * highest-ranked vectors, the same set in every head): for every segment copy
 * the len top-ranked rows of K and V, in ascending prompt position, into the
 * packed cache, and fill
 * row_offset / len / cap.  Segments whose rows would pass total_cap_rows raise
 * PKV_DEV_CAPACITY and copy nothing.
 *   k, v    [B,L,H,N,D] with strides, as for prefixkv_score
 *   order   [B,L,N], len [B,L] from prefixkv_search / prefixkv_apply_lengths
 *   kept    [B,L,N] int32 out, may be NULL (then workspace holds it): the
 *           retained positions in ascending order, first len entries valid
 */
int prefixkv_compact(const pkv_shape *shape, const void *k, pkv_strides ks, const void *v,
                     pkv_strides vs, const int32_t *order, const int32_t *len,
                     pkv_cache *cache, int32_t *kept, int32_t *dev_status, void *ws,
                     size_t ws_bytes, void *cuda_stream);

/*
 * Compression with cache merging (Sec. 4.3, paragraph "Eviction or merging", Tab. "merge"):
 * as prefixkv_compact, but a pruned vector is averaged into one retained vector instead of
 * being dropped.  Per layer and head, each pruned key k^m is matched to the retained key k^n
 * with the largest metric c^{mn}:
 *   PKV_MERGE_POSITION   c^{mn} = -|m - n|
 *   PKV_MERGE_FEATURE    c^{mn} = <k^m, k^n> / (|k^m| |k^n|)       (0 if a norm is 0)
 * and the cached key / value of n becomes the plain average of its own vector and of the
 * pruned vectors matched to it.  Where the paper is silent: the match is taken on the keys and
 * applied to the values too; among equal metrics the retained vector at the lower position
 * wins; averages are formed in fp32 and rounded once to the cache type.
 *   kept    as for prefixkv_compact
 *   match   [B,L,H,N] int32 out, may be NULL: for every position the index (into the
 *           segment's ascending retained list) of the row it was merged into; a retained
 *           position maps to its own row
 * prompt_len <= 4096; not combined with decode-time pruning (evict_distance must be 0).
 * Every prompt row of K and V is read once (not only the retained ones).
 */
enum { PKV_MERGE_POSITION = 1, PKV_MERGE_FEATURE = 2 };
int prefixkv_compact_merge(const pkv_shape *shape, const void *k, pkv_strides ks, const void *v,
                           pkv_strides vs, const int32_t *order, const int32_t *len,
                           pkv_cache *cache, int32_t mode, int32_t *kept, int32_t *match,
                           int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * One decode step over the ragged cache (Sec. 3.1: the newest token attends over
 * the cached key/value vectors): for every segment of layers [layer_begin,
 * layer_end), append k_new / v_new as row len, then
 *   out[b,l,h,:] = sum_j softmax_j(scale_l * <q[b,l,h], K_j[h]>) * V_j[h]
 * over all len + 1 rows, and set len += 1.
 *   q, k_new, v_new, out   [B,L,H,D] contiguous, dtype of the cache
 * A segment already at capacity raises PKV_DEV_CAPACITY, appends nothing and
 * writes zeros.
 * k_new and v_new may both be NULL: nothing is appended, len stays, and out attends over the
 * len rows that are there (a second query against the same cache).
 * With cache->evict_distance = d > 0 the layer proportions are kept while decoding (Sec. 3.1,
 * Fig. 2a; the distance and the exact rule are the cited work's, this is the reading): when
 * generated token g would push a layer past floor(len0 * (N + g + 1) / N) rows and token
 * g - d is still cached, the new row takes that token's slot and len stays; otherwise it is
 * appended.  Prompt rows are never dropped.  Calls on one cache, or sharing one workspace, must not overlap on
 * the GPU.
 * The call only enqueues kernels on cuda_stream, so it may be captured into a CUDA graph and
 * replayed once per token (same pointers, new contents); make one call on the device outside
 * any capture first, which sets the kernels up.
 */
int prefixkv_decode_attn(const pkv_shape *shape, pkv_cache *cache, const void *q,
                         const void *k_new, const void *v_new, const float *layer_scale,
                         int32_t layer_begin, int32_t layer_end, void *out,
                         int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The same decode step for callers that have no workspace to give.  (The paper
 * has no counterpart to this call; it exists for deployment.)
 *
 * Who needs it: a serving engine that claimed all free device memory for its
 * own pool when it started has nothing left for cudaMalloc to return once
 * requests arrive, and a runtime that must not stall between two tokens cannot
 * pay for cudaMalloc's implicit device-wide synchronisation.  Such callers
 * still pass every input and output; only the split-K scratch comes from the
 * library, as a fixed array of prefixkv_decode_static_limit_bytes() (16 MiB)
 * that each GPU holds from the moment it loads the library until the process
 * exits.
 *
 *  - The call allocates and frees nothing, on the device or through any
 *    library.
 *  - A shape whose scratch need, prefixkv_workspace_bytes(shape,
 *    PKV_WS_DECODE), is above the limit is refused with PKV_ERR_STATIC_LIMIT
 *    before anything is launched (prefixkv_last_cuda_error() then holds a
 *    sentence saying so); use prefixkv_decode_attn for those.
 *  - The first call on each device looks up the array's device address (that
 *    device must be current).  Make that first call during start-up, outside
 *    any stream capture.
 *  - All calls in the process, on any stream, share the one array per GPU, and
 *    it keeps whatever the previous call left.  The kernels write every slot
 *    before reading it, so nothing has to be cleared, but two calls that run
 *    on the same GPU at the same time overwrite each other's partial results:
 *    order them on one stream or with events.
 * Everything else (arguments, results, dev_status) is as for
 * prefixkv_decode_attn.
 */
size_t prefixkv_decode_static_limit_bytes(void);
int prefixkv_decode_attn_static(const pkv_shape *shape, pkv_cache *cache, const void *q,
                                const void *k_new, const void *v_new, const float *layer_scale,
                                int32_t layer_begin, int32_t layer_end, void *out,
                                int32_t *dev_status, void *cuda_stream);

/*
 * Lorenz-curve diagnostic of Sec. 3.2 / Fig. 3: Gini coefficient of each
 * segment's priority sequence from its cumulative sums (trapezoid rule).
 *   cum  [B,L,N] from prefixkv_search;  gini [B,L] fp64 out
 */
int prefixkv_gini(const pkv_shape *shape, const uint64_t *cum, double *gini, void *cuda_stream);

/*
 * Self-test of the bounded waits (a robustness aid; the paper has no counterpart).  Every
 * wait on an mbarrier inside the tensor-core scoring kernel (which = 0) and the streaming
 * decode kernel (which = 1) gives up after a fixed number of tries; the kernel then stops
 * waiting, finishes in bounds and reports.  This call runs that give-up path alone: one warp
 * waits, with a limit of a few thousand tries (milliseconds), on a barrier that nothing
 * completes, and dev_status[0] is raised to PKV_DEV_TIMEOUT.  Nothing faults or hangs.
 *   dev_status  [>= 1] int32, must hold PKV_DEV_OK on entry for the code to be recorded
 */
int prefixkv_selftest_bounded_wait(int32_t which, int32_t *dev_status, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PREFIXKV_H_ */

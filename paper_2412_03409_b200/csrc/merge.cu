// Cache merging (Sec. 4.3, "Eviction or merging", Tab. "merge"): compression after prefilling
// in which a pruned vector is not dropped but averaged into one retained vector.  For every
// layer and head each pruned key is matched to the retained key with the largest metric --
// minus the positional distance ("Position") or the cosine similarity of the two keys
// ("Feature") -- and a retained key / value is replaced by the plain average of itself and of
// the pruned ones matched to it.  Readings where the paper is silent: the match is taken on the
// keys and applied to the values too; equal metrics go to the retained vector at the lower
// position.
//
// One CTA per (segment, head).  The match of every position sits in shared memory; the
// similarities are FP32 FMA work (lane j of a warp owns retained key j of a 32-key tile that is
// staged transposed and pre-divided by its norm, the pruned key's channels are broadcast by
// shuffle): the contraction is small next to scoring and its argmax decides an integer, so it is
// kept in full fp32 rather than sent through bf16 tensor cores.  The averages are formed by a
// warp per retained row that walks the positions in ascending order, so the sums are
// reproducible bit for bit; every source row is read once (all N, not only the retained ones).
#include "common.cuh"

namespace pkv {

constexpr int kMergeMaxN = 4096;
constexpr int kMergeWarps = 8;

static size_t merge_smem_bytes(int N, int D)
{
    // retained list, match, best metric, reciprocal norms, one transposed tile of 32 retained keys
    return (size_t)N * (2 * sizeof(int32_t) + 2 * sizeof(float)) + (size_t)D * 33 * sizeof(float);
}

template <typename T, int D>
__global__ void __launch_bounds__(kMergeWarps * 32)
merge_rows_kernel(const T *__restrict__ k, pkv_strides ks, const T *__restrict__ v, pkv_strides vs,
                  const int32_t *__restrict__ kept, const int32_t *__restrict__ len,
                  const int64_t *__restrict__ row_offset, int L, int N, int H, int mode, T *__restrict__ ck,
                  T *__restrict__ cv, int32_t *__restrict__ match_out)
{
    constexpr int EPL = D / 32;  // channels per lane
    extern __shared__ __align__(16) unsigned char smem[];
    int32_t *s_kept = reinterpret_cast<int32_t *>(smem);     // [N] retained positions, ascending
    int32_t *s_match = s_kept + N;                           // [N] index into s_kept a position belongs to
    float *s_best = reinterpret_cast<float *>(s_match + N);  // [N] best metric so far (Feature)
    float *s_rnorm = s_best + N;                             // [N] 1 / |k| (0 for a zero key)
    float *s_kt = s_rnorm + N;                               // [D][33] retained keys of a tile, transposed, unit length
    const int h = blockIdx.x, seg = blockIdx.y;
    const int b = seg / L, l = seg % L;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    dependent_entry();  // the plan kernel's lists, lengths and offsets are complete
    const int n = len[seg];
    if (n <= 0) return;  // the segment did not fit the cache: reported by the plan kernel
    const T *kb = k + b * ks.b + l * ks.l + h * ks.h;
    const T *vb = v + b * vs.b + l * vs.l + h * vs.h;

    for (int m = tid; m < N; m += blockDim.x) {
        s_match[m] = -1;
        s_best[m] = -INFINITY;
    }
    for (int r = tid; r < n; r += blockDim.x) s_kept[r] = kept[(size_t)seg * N + r];
    __syncthreads();
    for (int r = tid; r < n; r += blockDim.x) s_match[s_kept[r]] = r;  // a retained position belongs to itself
    __syncthreads();

    if (mode == PKV_MERGE_POSITION) {
        // the nearest retained position, the lower one at equal distance
        for (int m = tid; m < N; m += blockDim.x) {
            if (s_match[m] >= 0) continue;
            int lo = 0, hi = n;  // first retained position above m
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (s_kept[mid] > m) hi = mid; else lo = mid + 1;
            }
            int r = lo;
            if (lo == n) r = n - 1;
            else if (lo > 0 && m - s_kept[lo - 1] <= s_kept[lo] - m) r = lo - 1;
            s_best[m] = 0.f;
            s_match[m] = r;
        }
    } else {
        // cosine similarity of the keys
        for (int p = warp; p < N; p += kMergeWarps) {
            float s = 0.f;
#pragma unroll
            for (int i = 0; i < EPL; ++i) {
                const float x = to_float(kb[(int64_t)p * ks.n + lane * EPL + i]);
                s = fmaf(x, x, s);
            }
            s = warp_sum(s);
            if (lane == 0) s_rnorm[p] = s > 0.f ? rsqrtf(s) : 0.f;
        }
        __syncthreads();
        for (int r0 = 0; r0 < n; r0 += 32) {
            // stage retained keys r0 .. r0 + 31, transposed and divided by their norms
            for (int idx = tid; idx < 32 * D; idx += blockDim.x) {
                const int j = idx / D, d = idx % D;
                float x = 0.f;
                if (r0 + j < n) {
                    const int pos = s_kept[r0 + j];
                    x = to_float(kb[(int64_t)pos * ks.n + d]) * s_rnorm[pos];
                }
                s_kt[d * 33 + j] = x;
            }
            __syncthreads();
            for (int m = warp; m < N; m += kMergeWarps) {
                if (s_best[m] == -INFINITY && s_match[m] >= 0) continue;  // a retained position
                float km[EPL];
#pragma unroll
                for (int i = 0; i < EPL; ++i) km[i] = to_float(kb[(int64_t)m * ks.n + i * 32 + lane]);
                float c = 0.f;
#pragma unroll
                for (int i = 0; i < EPL; ++i)
#pragma unroll 8
                    for (int dd = 0; dd < 32; ++dd)
                        c = fmaf(__shfl_sync(0xffffffffu, km[i], dd), s_kt[(i * 32 + dd) * 33 + lane], c);
                c *= s_rnorm[m];  // (a zero pruned key: every metric is 0 and the first retained key wins)
                if (r0 + lane >= n) c = -INFINITY;
                // largest metric of the tile, lowest lane among equals
                float bc = c;
                int bj = lane;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float oc = __shfl_xor_sync(0xffffffffu, bc, o);
                    const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
                    if (oc > bc || (oc == bc && oj < bj)) {
                        bc = oc;
                        bj = oj;
                    }
                }
                if (lane == 0 && bc > s_best[m]) {  // strict: an equal metric in a later tile (higher position) loses
                    s_best[m] = bc;
                    s_match[m] = r0 + bj;
                }
            }
            __syncthreads();
        }
    }
    __syncthreads();
    if (match_out)
        for (int m = tid; m < N; m += blockDim.x) match_out[((size_t)seg * H + h) * N + m] = s_match[m];

    // Averages: a warp per retained row, positions in ascending order.
    const int64_t off = row_offset[seg];
    for (int r = warp; r < n; r += kMergeWarps) {
        float ak[EPL], av[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) ak[i] = av[i] = 0.f;
        int count = 0;
        for (int m0 = 0; m0 < N; m0 += 32) {
            const int m = m0 + lane;
            unsigned members = __ballot_sync(0xffffffffu, m < N && s_match[m] == r);
            while (members) {
                const int p = m0 + __ffs(members) - 1;
                members &= members - 1;
                ++count;
#pragma unroll
                for (int i = 0; i < EPL; ++i) {
                    ak[i] += to_float(kb[(int64_t)p * ks.n + lane * EPL + i]);
                    av[i] += to_float(vb[(int64_t)p * vs.n + lane * EPL + i]);
                }
            }
        }
        const float inv = 1.f / (float)count;  // count >= 1: the retained row itself
        T *dk = ck + ((size_t)(off + r) * H + h) * D + lane * EPL;
        T *dv = cv + ((size_t)(off + r) * H + h) * D + lane * EPL;
#pragma unroll
        for (int i = 0; i < EPL; ++i) {
            dk[i] = from_float<T>(ak[i] * inv);
            dv[i] = from_float<T>(av[i] * inv);
        }
    }
}

// The plan kernel of the compaction (row offsets, lengths, capacities, ascending retained lists).
cudaError_t launch_compact_plan(const pkv_shape *shape, const int32_t *order, const int32_t *len, pkv_cache *cache,
                                int32_t *kept, int32_t *dev_status, cudaStream_t stream);

template <typename T, int D>
static int launch_merge(const pkv_shape *s, const void *k, pkv_strides ks, const void *v, pkv_strides vs,
                        const int32_t *kept, pkv_cache *c, int mode, int32_t *match, cudaStream_t st)
{
    static bool done[64] = {};
    const size_t smem = merge_smem_bytes(s->prompt_len, D);
    int rc = ensure_dynamic_smem((const void *)merge_rows_kernel<T, D>, (int)merge_smem_bytes(kMergeMaxN, D), done);
    if (rc != PKV_OK) return rc;
    cudaError_t e = launch_dependent(merge_rows_kernel<T, D>, dim3(s->heads, s->batch * s->layers), dim3(kMergeWarps * 32),
                                     smem, st, (const T *)k, ks, (const T *)v, vs, kept, (const int32_t *)c->len,
                                     (const int64_t *)c->row_offset, (int)s->layers, (int)s->prompt_len, (int)s->heads,
                                     mode, (T *)c->k, (T *)c->v, match);
    if (e != cudaSuccess) {
        set_cuda_error(e, "merge_rows_kernel");
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

}  // namespace pkv

using namespace pkv;

extern "C" int prefixkv_compact_merge(const pkv_shape *shape, const void *k, pkv_strides ks, const void *v,
                                      pkv_strides vs, const int32_t *order, const int32_t *len, pkv_cache *cache,
                                      int32_t mode, int32_t *kept, int32_t *match, int32_t *dev_status, void *ws,
                                      size_t ws_bytes, void *cuda_stream)
{
    if (!shape_ok(shape) || !k || !v || !order || !len || !cache || !cache->k || !cache->v || !cache->row_offset ||
        !cache->len || !cache->cap || cache->decode_cap < 0 || cache->total_cap_rows <= 0 || !dev_status ||
        (mode != PKV_MERGE_POSITION && mode != PKV_MERGE_FEATURE))
        return PKV_ERR_INVALID_ARG;
    if (!shape_supported(shape) || shape->prompt_len > kMergeMaxN) return PKV_ERR_UNSUPPORTED;
    if (cache->evict_distance != 0) return PKV_ERR_UNSUPPORTED;  // decode-time pruning starts from a plain compaction
    const int per16 = 16 / (int)esize(shape);
    int64_t st[8] = {ks.b, ks.l, ks.h, ks.n, vs.b, vs.l, vs.h, vs.n};
    for (int i = 0; i < 8; ++i)
        if (st[i] < 0 || st[i] % per16 != 0) return PKV_ERR_INVALID_ARG;
    if (!aligned(k, 16) || !aligned(v, 16) || !aligned(cache->k, 16) || !aligned(cache->v, 16))
        return PKV_ERR_INVALID_ARG;
    if ((size_t)shape->batch * shape->layers > 65535) return PKV_ERR_UNSUPPORTED;
    if (!kept) {
        size_t need = (size_t)shape->batch * shape->layers * shape->prompt_len * sizeof(int32_t);
        if (!ws || !aligned(ws, kWsAlign) || ws_bytes < need) return PKV_ERR_WORKSPACE;
        kept = (int32_t *)ws;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    cudaError_t e = launch_compact_plan(shape, order, len, cache, kept, dev_status, stream);
    if (e != cudaSuccess) {
        set_cuda_error(e, "compact_plan_kernel");
        return PKV_ERR_CUDA;
    }
#define PKV_MERGE(T, DD) return launch_merge<T, DD>(shape, k, ks, v, vs, kept, cache, mode, match, stream)
    if (shape->dtype == PKV_F32) {
        if (shape->head_dim == 64) PKV_MERGE(float, 64);
        PKV_MERGE(float, 128);
    }
    if (shape->head_dim == 64) PKV_MERGE(__nv_bfloat16, 64);
    PKV_MERGE(__nv_bfloat16, 128);
#undef PKV_MERGE
}

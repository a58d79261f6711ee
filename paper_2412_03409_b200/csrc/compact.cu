// Compression after prefilling (Sec. 3.1, Fig. 2a): the len top-ranked rows of
// every segment are copied, in ascending prompt position, into one packed
// ragged cache.  Pure data movement in 16-byte vectors; HBM-bound.
#include "common.cuh"

namespace pkv {

// One CTA per segment: row offset of the segment (exclusive sum of capacities of
// the segments before it), capacity check, and the ascending list of retained
// positions (a bitmap over positions filled from the first len ranks, then a
// scan over word popcounts).
__global__ void __launch_bounds__(1024)
compact_plan_kernel(const int32_t *__restrict__ order, const int32_t *__restrict__ len_in, int nseg,
                    int L, int N, int decode_cap, int64_t total_cap_rows,
                    int64_t *__restrict__ row_offset, int32_t *__restrict__ len_out,
                    int32_t *__restrict__ cap_out, int32_t *__restrict__ kept, int32_t *dev_status,
                    int32_t *len0, int32_t *gen, int32_t *slot_ring, int ring_size)
{
    __shared__ uint32_t bitmap[kMaxPromptLen / 32];
    __shared__ int64_t red[32];
    __shared__ int wsum[32];
    __shared__ int64_t s_off;
    const int seg = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = seg / L;
    dependent_entry();

    auto clamp_len = [&](int v) { return (v < 1 || v > N) ? 0 : v; };

    // offset = sum over earlier segments of (len + decode_cap)
    int64_t part = 0;
    for (int s = tid; s < seg; s += blockDim.x) part += (int64_t)clamp_len(len_in[s]) + decode_cap;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) red[warp] = part;
    for (int i = tid; i < kMaxPromptLen / 32; i += blockDim.x) bitmap[i] = 0;
    __syncthreads();
    if (warp == 0) {
        int64_t t = (lane < (blockDim.x >> 5)) ? red[lane] : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0) s_off = t;
    }
    __syncthreads();
    const int64_t off = s_off;
    int raw = len_in[seg];
    int n = clamp_len(raw);
    int cap = n + decode_cap;
    bool fits = off + cap <= total_cap_rows;
    if (tid == 0) {
        if (raw != n) raise_status(dev_status, b, PKV_DEV_BAD_LENGTH);
        if (!fits) raise_status(dev_status, b, PKV_DEV_CAPACITY);
        row_offset[seg] = off;
        if (seg == nseg - 1) row_offset[nseg] = off + cap;
        len_out[seg] = fits ? n : 0;
        cap_out[seg] = fits ? cap : 0;
        if (len0) len0[seg] = fits ? n : 0;
        if (gen) gen[seg] = 0;
    }
    if (slot_ring)
        for (int i = tid; i < ring_size; i += blockDim.x) slot_ring[(size_t)seg * ring_size + i] = -1;
    if (!fits) n = 0;

    const int32_t *ord = order + (size_t)seg * N;
    for (int j = tid; j < n; j += blockDim.x) {
        int pos = ord[j];
        if (pos >= 0 && pos < N) atomicOr(&bitmap[pos >> 5], 1u << (pos & 31));
    }
    __syncthreads();
    const int nwords = (N + 31) >> 5;  // <= 512 <= blockDim.x
    uint32_t word = tid < nwords ? bitmap[tid] : 0;
    int cnt = __popc(word), incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int t = wsum[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int up = __shfl_up_sync(0xffffffffu, t, o);
            if (lane >= o) t += up;
        }
        wsum[lane] = t;
    }
    __syncthreads();
    int dst = incl - cnt + (warp ? wsum[warp - 1] : 0);
    int32_t *out = kept + (size_t)seg * N;
    while (word) {
        int bit = __ffs(word) - 1;
        word &= word - 1;
        if (dst < n) out[dst] = tid * 32 + bit;
        ++dst;
    }
}

// grid (segments, row slices); each CTA copies whole rows (K and V, all heads).
template <int VEC_PER_HEAD>
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4 *__restrict__ k, const uint4 *__restrict__ v, pkv_strides ks16,
                   pkv_strides vs16, const int32_t *__restrict__ kept,
                   const int32_t *__restrict__ len, const int64_t *__restrict__ row_offset, int L,
                   int N, int H, uint4 *__restrict__ ck, uint4 *__restrict__ cv)
{
    const int seg = blockIdx.x;
    dependent_entry();  // the plan kernel's lists, lengths and offsets are complete
    const int n = len[seg];
    const int b = seg / L, l = seg % L;
    const int64_t off = row_offset[seg];
    const int row_vecs = H * VEC_PER_HEAD;
    const uint4 *kb = k + b * ks16.b + l * ks16.l;
    const uint4 *vb = v + b * vs16.b + l * vs16.l;
    const int32_t *kp = kept + (size_t)seg * N;
    for (int r = blockIdx.y; r < n; r += gridDim.y) {
        const int pos = kp[r];
        uint4 *dk = ck + (off + r) * row_vecs;
        uint4 *dv = cv + (off + r) * row_vecs;
        for (int x = threadIdx.x; x < row_vecs; x += 256 * 2) {
            int x1 = x + 256;
            int h0 = x / VEC_PER_HEAD, c0 = x % VEC_PER_HEAD;
            int h1 = x1 / VEC_PER_HEAD, c1 = x1 % VEC_PER_HEAD;
            bool two = x1 < row_vecs;
            uint4 a0 = __ldg(kb + h0 * ks16.h + pos * ks16.n + c0);
            uint4 b0 = __ldg(vb + h0 * vs16.h + pos * vs16.n + c0);
            uint4 a1, b1;
            if (two) {
                a1 = __ldg(kb + h1 * ks16.h + pos * ks16.n + c1);
                b1 = __ldg(vb + h1 * vs16.h + pos * vs16.n + c1);
            }
            dk[x] = a0;
            dv[x] = b0;
            if (two) {
                dk[x1] = a1;
                dv[x1] = b1;
            }
        }
    }
}

cudaError_t launch_compact_plan(const pkv_shape *shape, const int32_t *order, const int32_t *len, pkv_cache *cache,
                                int32_t *kept, int32_t *dev_status, cudaStream_t stream)
{
    const int nseg = shape->batch * shape->layers;
    const bool pruning = cache->evict_distance > 0;
    return launch_dependent(compact_plan_kernel, dim3(nseg), dim3(1024), 0, stream, order, len, nseg, (int)shape->layers,
                            (int)shape->prompt_len, cache->decode_cap, cache->total_cap_rows, cache->row_offset,
                            cache->len, cache->cap, kept, dev_status, pruning ? cache->len0 : nullptr,
                            pruning ? cache->gen : nullptr, pruning ? cache->slot_ring : nullptr,
                            cache->evict_distance + 1);
}

}  // namespace pkv

using namespace pkv;

extern "C" int prefixkv_compact(const pkv_shape *shape, const void *k, pkv_strides ks,
                                const void *v, pkv_strides vs, const int32_t *order,
                                const int32_t *len, pkv_cache *cache, int32_t *kept,
                                int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!shape_ok(shape) || !k || !v || !order || !len || !cache || !cache->k || !cache->v ||
        !cache->row_offset || !cache->len || !cache->cap || cache->decode_cap < 0 ||
        cache->total_cap_rows <= 0 || !dev_status)
        return PKV_ERR_INVALID_ARG;
    if (!shape_supported(shape)) return PKV_ERR_UNSUPPORTED;
    const int B = shape->batch, L = shape->layers, N = shape->prompt_len, H = shape->heads;
    const size_t es = esize(shape);
    const int per16 = 16 / (int)es;  // elements per 16-byte vector
    int64_t st[8] = {ks.b, ks.l, ks.h, ks.n, vs.b, vs.l, vs.h, vs.n};
    for (int i = 0; i < 8; ++i)
        if (st[i] < 0 || st[i] % per16 != 0) return PKV_ERR_INVALID_ARG;
    if (!aligned(k, 16) || !aligned(v, 16) || !aligned(cache->k, 16) || !aligned(cache->v, 16))
        return PKV_ERR_INVALID_ARG;
    const int nseg = B * L;
    if (!kept) {
        size_t need = (size_t)nseg * N * sizeof(int32_t);
        if (!ws || !aligned(ws, kWsAlign) || ws_bytes < need) return PKV_ERR_WORKSPACE;
        kept = (int32_t *)ws;
    }
    if (cache->evict_distance < 0) return PKV_ERR_INVALID_ARG;
    const bool pruning = cache->evict_distance > 0;
    if (pruning && (!cache->len0 || !cache->gen || !cache->slot_ring)) return PKV_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    cudaError_t e = launch_compact_plan(shape, order, len, cache, kept, dev_status, stream);
    if (e != cudaSuccess) {
        set_cuda_error(e, "compact_plan_kernel");
        return PKV_ERR_CUDA;
    }

    pkv_strides k16 = {ks.b / per16, ks.l / per16, ks.h / per16, ks.n / per16};
    pkv_strides v16 = {vs.b / per16, vs.l / per16, vs.h / per16, vs.n / per16};
    const int vph = shape->head_dim / per16;
    int slices = (148 * 8 + nseg - 1) / nseg;
    if (slices < 1) slices = 1;
    if (slices > N) slices = N;
    dim3 grid(nseg, slices);
#define PKV_GATHER(V)                                                                                  \
    e = launch_dependent(gather_rows_kernel<V>, grid, dim3(256), 0, stream, (const uint4 *)k,          \
                         (const uint4 *)v, k16, v16, (const int32_t *)kept, (const int32_t *)cache->len, \
                         (const int64_t *)cache->row_offset, L, N, H, (uint4 *)cache->k, (uint4 *)cache->v)
    switch (vph) {
    case 8: PKV_GATHER(8); break;
    case 16: PKV_GATHER(16); break;
    case 32: PKV_GATHER(32); break;
    default: return PKV_ERR_UNSUPPORTED;
    }
#undef PKV_GATHER
    if (e != cudaSuccess) {
        set_cuda_error(e, "gather_rows_kernel");
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

// Decode attention over the ragged per-layer cache (Sec. 3.1, Fig. 2a): the
// newest token's key/value row is appended to every segment, then its query
// attends over all rows of the segment.  One byte of K/V is read per ~1 FLOP, so
// the kernel is HBM-bound and runs on plain FP32 ALUs with an fp32 softmax.
//
// Split-K: a segment's rows are cut into `splits` slices handled by different
// CTAs; each writes an un-normalised partial (running max, sum, accumulator)
// to workspace and a second kernel merges them and bumps len.
#include "common.cuh"

namespace pkv {

constexpr float kLog2e = 1.4426950408889634f;

template <typename T, int EPL>
__device__ __forceinline__ void load_frag(const T *p, int lane, float (&x)[EPL]);

template <> __device__ __forceinline__ void load_frag<float, 2>(const float *p, int lane, float (&x)[2])
{
    float2 t = *reinterpret_cast<const float2 *>(p + lane * 2);
    x[0] = t.x; x[1] = t.y;
}
template <> __device__ __forceinline__ void load_frag<float, 4>(const float *p, int lane, float (&x)[4])
{
    float4 t = *reinterpret_cast<const float4 *>(p + lane * 4);
    x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
}
template <>
__device__ __forceinline__ void load_frag<__nv_bfloat16, 2>(const __nv_bfloat16 *p, int lane, float (&x)[2])
{
    uint32_t raw = *reinterpret_cast<const uint32_t *>(p + lane * 2);
    x[0] = __uint_as_float(raw << 16); x[1] = __uint_as_float(raw & 0xffff0000u);
}
template <>
__device__ __forceinline__ void load_frag<__nv_bfloat16, 4>(const __nv_bfloat16 *p, int lane, float (&x)[4])
{
    uint2 raw = *reinterpret_cast<const uint2 *>(p + lane * 4);
    x[0] = __uint_as_float(raw.x << 16); x[1] = __uint_as_float(raw.x & 0xffff0000u);
    x[2] = __uint_as_float(raw.y << 16); x[3] = __uint_as_float(raw.y & 0xffff0000u);
}

template <typename T, int EPL>
__device__ __forceinline__ void store_frag(T *p, int lane, const float (&x)[EPL])
{
#pragma unroll
    for (int i = 0; i < EPL; ++i) p[lane * EPL + i] = from_float<T>(x[i]);
}

// grid (splits, active segments); 8 warps, warp w takes heads w, w+8, ...
template <typename T, int D>
__global__ void __launch_bounds__(256)
decode_partial_kernel(const T *__restrict__ q, const T *__restrict__ k_new, const T *__restrict__ v_new,
                      T *__restrict__ ck, T *__restrict__ cv, const int64_t *__restrict__ row_offset,
                      const int32_t *__restrict__ len, const int32_t *__restrict__ cap,
                      const float *__restrict__ layer_scale, int L, int H, int layer_begin, int nl,
                      float *__restrict__ part_acc, float *__restrict__ part_ml, int32_t *dev_status)
{
    constexpr int EPL = D / 32;
    const int sp = blockIdx.x, splits = gridDim.x;
    const int b = blockIdx.y / nl, l = layer_begin + blockIdx.y % nl;
    const int seg = b * L + l;
    const int n = len[seg];
    if (n < 1 || n + 1 > cap[seg]) {  // never compacted, or full: reported, zero output, length kept
        if (threadIdx.x == 0 && sp == 0) raise_status(dev_status, b, PKV_DEV_CAPACITY);
        return;
    }
    const int rows = n + 1;
    const int chunk = (rows + splits - 1) / splits;
    const int r0 = sp * chunk;
    const int r1 = min(rows, r0 + chunk);
    const int64_t off = row_offset[seg];
    const float sc = layer_scale[l] * kLog2e;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for (int h = warp; h < H; h += 8) {
        const size_t qoff = ((size_t)seg * H + h) * D;
        float qf[EPL];
        load_frag<T, EPL>(q + qoff, lane, qf);
#pragma unroll
        for (int i = 0; i < EPL; ++i) qf[i] *= sc;
        float m = -INFINITY, lsum = 0.f, acc[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] = 0.f;
        for (int r = r0; r < r1; ++r) {
            float kf[EPL], vf[EPL];
            T *krow = ck + ((size_t)(off + r) * H + h) * D;
            T *vrow = cv + ((size_t)(off + r) * H + h) * D;
            if (r == n) {  // the row being appended this step
                load_frag<T, EPL>(k_new + qoff, lane, kf);
                load_frag<T, EPL>(v_new + qoff, lane, vf);
                store_frag<T, EPL>(krow, lane, kf);
                store_frag<T, EPL>(vrow, lane, vf);
            } else {
                load_frag<T, EPL>(krow, lane, kf);
                load_frag<T, EPL>(vrow, lane, vf);
            }
            float s = 0.f;
#pragma unroll
            for (int i = 0; i < EPL; ++i) s = fmaf(qf[i], kf[i], s);
            s = warp_sum(s);
            float mn = fmaxf(m, s);
            float corr = exp2f(m - mn), p = exp2f(s - mn);
            lsum = lsum * corr + p;
#pragma unroll
            for (int i = 0; i < EPL; ++i) acc[i] = acc[i] * corr + p * vf[i];
            m = mn;
        }
        const size_t po = ((size_t)blockIdx.y * splits + sp) * H + h;
        float *pa = part_acc + po * D;
#pragma unroll
        for (int i = 0; i < EPL; ++i) pa[lane * EPL + i] = acc[i];
        if (lane == 0) {
            part_ml[po * 2] = m;
            part_ml[po * 2 + 1] = lsum;
        }
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(256)
decode_merge_kernel(const float *__restrict__ part_acc, const float *__restrict__ part_ml, int splits,
                    int32_t *__restrict__ len, const int32_t *__restrict__ cap, int L, int H,
                    int layer_begin, int nl, T *__restrict__ out)
{
    constexpr int EPL = D / 32;
    const int b = blockIdx.x / nl, l = layer_begin + blockIdx.x % nl;
    const int seg = b * L + l;
    const int n = len[seg];
    const bool full = n < 1 || n + 1 > cap[seg];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int h = warp; h < H; h += 8) {
        float o[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) o[i] = 0.f;
        if (!full) {
            float M = -INFINITY;
            for (int sp = 0; sp < splits; ++sp)
                M = fmaxf(M, part_ml[(((size_t)blockIdx.x * splits + sp) * H + h) * 2]);
            float z = 0.f;
            for (int sp = 0; sp < splits; ++sp) {
                const size_t po = ((size_t)blockIdx.x * splits + sp) * H + h;
                float w = exp2f(part_ml[po * 2] - M);
                z += w * part_ml[po * 2 + 1];
#pragma unroll
                for (int i = 0; i < EPL; ++i) o[i] += w * part_acc[po * D + lane * EPL + i];
            }
            float inv = 1.f / z;
#pragma unroll
            for (int i = 0; i < EPL; ++i) o[i] *= inv;
        }
        store_frag<T, EPL>(out + ((size_t)seg * H + h) * D, lane, o);
    }
    __syncthreads();
    if (threadIdx.x == 0 && !full) len[seg] = n + 1;
}

static int pick_splits(int nseg_active)
{
    int s = (148 * 4 + nseg_active - 1) / nseg_active;
    return s < 1 ? 1 : (s > 64 ? 64 : s);
}

size_t decode_stream_ws_bytes(const pkv_shape *s);
size_t decode_heads_ws_bytes();
int launch_decode_heads(const pkv_shape *s, pkv_cache *c, const void *q, const void *kn, const void *vn,
                        const float *scale, int lb, int le, void *out, int32_t *dev_status, void *ws, cudaStream_t st);
int launch_decode_stream(const pkv_shape *s, pkv_cache *c, const void *q, const void *kn,
                         const void *vn, const float *scale, int lb, int le, void *out,
                         int32_t *dev_status, void *ws, cudaStream_t st);

size_t decode_ws_bytes(const pkv_shape *s)
{
    // Two-kernel path: splits * active segments never exceeds 148 * 4 + B * L partial slots.
    size_t nseg = (size_t)s->batch * s->layers;
    size_t slots = 148 * 4 + nseg;
    size_t per = (size_t)s->heads * (s->head_dim + 2) * sizeof(float);
    size_t two = round_up(slots * per, kWsAlign), one = decode_stream_ws_bytes(s), heads = decode_heads_ws_bytes();
    size_t need = two > one ? two : one;
    return need > heads ? need : heads;
}

template <typename T, int D>
static int launch_decode(const pkv_shape *s, pkv_cache *c, const void *q, const void *kn,
                         const void *vn, const float *scale, int lb, int le, void *out,
                         int32_t *dev_status, void *ws, cudaStream_t st)
{
    const int nl = le - lb, nact = s->batch * nl, H = s->heads;
    const int splits = pick_splits(nact);
    float *part_acc = (float *)ws;
    float *part_ml = part_acc + (size_t)nact * splits * H * D;
    dim3 grid(splits, nact);
    decode_partial_kernel<T, D><<<grid, 256, 0, st>>>(
        (const T *)q, (const T *)kn, (const T *)vn, (T *)c->k, (T *)c->v, c->row_offset, c->len,
        c->cap, scale, s->layers, H, lb, nl, part_acc, part_ml, dev_status);
    int rc = check_launch("decode_partial_kernel");
    if (rc != PKV_OK) return rc;
    decode_merge_kernel<T, D><<<nact, 256, 0, st>>>(part_acc, part_ml, splits, c->len, c->cap,
                                                    s->layers, H, lb, nl, (T *)out);
    return check_launch("decode_merge_kernel");
}

}  // namespace pkv

using namespace pkv;

extern "C" int prefixkv_decode_attn(const pkv_shape *shape, pkv_cache *cache, const void *q,
                                    const void *k_new, const void *v_new, const float *layer_scale,
                                    int32_t layer_begin, int32_t layer_end, void *out,
                                    int32_t *dev_status, void *ws, size_t ws_bytes,
                                    void *cuda_stream)
{
    if (!shape_ok(shape) || !cache || !cache->k || !cache->v || !cache->row_offset || !cache->len ||
        !cache->cap || !q || (k_new == nullptr) != (v_new == nullptr) || !layer_scale || !out || !dev_status)
        return PKV_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_end > shape->layers || layer_begin >= layer_end)
        return PKV_ERR_INVALID_ARG;
    if (cache->evict_distance < 0 ||
        (cache->evict_distance > 0 && (!cache->len0 || !cache->gen || !cache->slot_ring)))
        return PKV_ERR_INVALID_ARG;
    if (!shape_supported(shape)) return PKV_ERR_UNSUPPORTED;
    if (!aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(out, 16) ||
        !aligned(cache->k, 16) || !aligned(cache->v, 16))
        return PKV_ERR_INVALID_ARG;
    if ((size_t)shape->batch * (layer_end - layer_begin) > 65535) return PKV_ERR_UNSUPPORTED;
    if (!ws || !aligned(ws, kWsAlign) || ws_bytes < decode_ws_bytes(shape)) return PKV_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    {
        // Few segments: whole (segment, head) items per CTA, no partials and no second kernel.
        int rc = launch_decode_heads(shape, cache, q, k_new, v_new, layer_scale, layer_begin, layer_end, out, dev_status,
                                     ws, st);
        if (rc >= 0) return rc;  // -1: not a case for that kernel
    }
    {
        // The streaming kernel plans at most 1024 segments at a time: a larger batch x layer range
        // goes through it in layer chunks, one launch after the other on the stream.
        const int max_active = 1024;
        int step = layer_end - layer_begin;
        if ((size_t)shape->batch * step > (size_t)max_active && shape->batch <= max_active)
            step = max_active / shape->batch;
        int rc = -1;
        for (int lb = layer_begin; lb < layer_end; lb += step) {
            const int le = lb + step < layer_end ? lb + step : layer_end;
            rc = launch_decode_stream(shape, cache, q, k_new, v_new, layer_scale, lb, le, out, dev_status, ws, st);
            if (rc != PKV_OK) break;
        }
        if (rc >= 0) return rc;  // -1: shape outside the streaming kernel, use the two-kernel path
    }
    if (cache->evict_distance != 0) return PKV_ERR_UNSUPPORTED;  // pruning lives in the streaming kernel
    if (!k_new) return PKV_ERR_UNSUPPORTED;                       // and so does attending without appending
#define PKV_DEC(T, D)                                                                              \
    return launch_decode<T, D>(shape, cache, q, k_new, v_new, layer_scale, layer_begin, layer_end, \
                               out, dev_status, ws, st)
    if (shape->dtype == PKV_F32) {
        if (shape->head_dim == 64) PKV_DEC(float, 64);
        PKV_DEC(float, 128);
    } else {
        if (shape->head_dim == 64) PKV_DEC(__nv_bfloat16, 64);
        PKV_DEC(__nv_bfloat16, 128);
    }
#undef PKV_DEC
}

// ---------------------------------------------------------------------------
// Decode step for callers that cannot hand over workspace.
//
// Some callers of this library are not able to obtain device memory when they
// reach the decode loop: a serving engine that gave every free byte to its own
// pool at start-up has nothing left for cudaMalloc to return, and a runtime that
// must never stall cannot afford cudaMalloc's implicit device-wide
// synchronisation between two tokens.  For them the split-K partials live in a
// fixed device array that is part of the library image: every GPU that loads
// the library carries kStaticScratchBytes for it until the process exits.
//
// In host code the array's name only stands for the symbol; it is not a device
// address.  The real address is looked up once per device with
// cudaGetSymbolAddress (while that device is current) and handed to the same
// kernels the workspace entry point launches.
// ---------------------------------------------------------------------------
#include <mutex>

namespace pkv {

constexpr size_t kStaticScratchBytes = 16u << 20;  // 16 MiB per GPU
static __device__ __align__(256) unsigned char g_decode_scratch[kStaticScratchBytes];

static int static_scratch_address(void **out)
{
    static std::mutex mu;
    static void *addr[64] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        set_cuda_error(e, "cudaGetDevice");
        return PKV_ERR_CUDA;
    }
    if (dev < 0 || dev >= 64) {
        set_cuda_error(cudaErrorInvalidDevice, "static scratch: device index above 63");
        return PKV_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_decode_scratch);
        if (e != cudaSuccess || !p) {
            set_cuda_error(e, "cudaGetSymbolAddress(decode scratch)");
            return PKV_ERR_CUDA;
        }
        addr[dev] = p;
    }
    *out = addr[dev];
    return PKV_OK;
}

}  // namespace pkv

extern "C" size_t prefixkv_decode_static_limit_bytes(void) { return pkv::kStaticScratchBytes; }

extern "C" int prefixkv_decode_attn_static(const pkv_shape *shape, pkv_cache *cache, const void *q,
                                           const void *k_new, const void *v_new,
                                           const float *layer_scale, int32_t layer_begin,
                                           int32_t layer_end, void *out, int32_t *dev_status,
                                           void *cuda_stream)
{
    if (!shape_ok(shape)) return PKV_ERR_INVALID_ARG;
    if (!shape_supported(shape)) return PKV_ERR_UNSUPPORTED;
    const size_t need = decode_ws_bytes(shape);
    if (need > kStaticScratchBytes) {
        set_error_text("prefixkv_decode_attn_static: this shape needs more scratch than the "
                       "built-in 16 MiB array; use prefixkv_decode_attn with caller workspace");
        return PKV_ERR_STATIC_LIMIT;
    }
    void *scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != PKV_OK) return rc;
    return prefixkv_decode_attn(shape, cache, q, k_new, v_new, layer_scale, layer_begin, layer_end,
                                out, dev_status, scratch, kStaticScratchBytes, cuda_stream);
}

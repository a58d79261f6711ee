// Host-side glue of the C ABI: error record, workspace sizing, score dispatch,
// and the Lorenz/Gini diagnostic.
#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace pkv {

static thread_local char g_err[256] = "";

void set_cuda_error(cudaError_t e, const char *where)
{
    snprintf(g_err, sizeof(g_err), "%s: %s", where, cudaGetErrorString(e));
}

void set_error_text(const char *text) { snprintf(g_err, sizeof(g_err), "%s", text); }

int check_launch(const char *where)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_cuda_error(e, where);
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

int ensure_dynamic_smem(const void *func, int bytes, bool *done_per_device)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        set_cuda_error(e, "cudaGetDevice");
        return PKV_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64 && done_per_device[dev]) return PKV_OK;
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) {
        set_cuda_error(e, "cudaFuncSetAttribute(max dynamic shared memory)");
        return PKV_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) done_per_device[dev] = true;
    return PKV_OK;
}

size_t decode_ws_bytes(const pkv_shape *s);

template <typename T, int D>
int launch_score_simt(const pkv_shape *s, const void *q, pkv_strides qs, const void *k,
                      pkv_strides ks, const float *scale, const float *lse, float *scores,
                      void *ws, cudaStream_t st);

int launch_score_tc(const pkv_shape *s, const void *q, pkv_strides qs, const void *k,
                    pkv_strides ks, const float *scale, const float *lse, float *scores, void *ws,
                    cudaStream_t st);
bool score_tc_usable(const pkv_shape *s, const void *q, pkv_strides qs, const void *k, pkv_strides ks);

size_t score_tc_ws_bytes(const pkv_shape *s);
int selftest_wait_score(int32_t *dev_status, cudaStream_t st);
int selftest_wait_stream(int32_t *dev_status, cudaStream_t st);

static size_t score_ws_bytes(const pkv_shape *s)
{
    // per-head column sums + per-query log-sum-exp, both [B, L, H, N] fp32; the tensor-core
    // path pads the second to whole 128-query tiles
    size_t per = (size_t)s->batch * s->layers * s->heads * s->prompt_len * sizeof(float);
    size_t simt = round_up(2 * per, kWsAlign), tc = score_tc_ws_bytes(s);
    return simt > tc ? simt : tc;
}

// Gini coefficient from the descending cumulative sums.  The Lorenz curve over
// the ascending order has ordinate (total - cum[N-1-k]) / total after k rows;
// the area under it is summed by trapezoids.
__global__ void gini_kernel(const uint64_t *__restrict__ cum, int N, double *__restrict__ gini)
{
    __shared__ double red[32];
    const uint64_t *c = cum + (size_t)blockIdx.x * N;
    const double total = (double)c[N - 1];
    double area = 0.0;
    for (int k = threadIdx.x; k < N; k += blockDim.x) {
        double lo = total - (double)c[N - 1 - k];
        double hi = (k + 1 < N) ? total - (double)c[N - 2 - k] : total;
        area += lo + hi;
    }
    for (int o = 16; o > 0; o >>= 1) area += __shfl_xor_sync(0xffffffffu, area, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = area;
    __syncthreads();
    if (threadIdx.x < 32) {
        double t = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.0;
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (threadIdx.x == 0)
            gini[blockIdx.x] = total > 0.0 ? 1.0 - t / (total * (double)N) : 0.0;
    }
}

}  // namespace pkv

using namespace pkv;

extern "C" const char *prefixkv_last_cuda_error(void) { return g_err; }

extern "C" size_t prefixkv_workspace_bytes(const pkv_shape *shape, int which)
{
    if (!shape_ok(shape) || !shape_supported(shape)) return 0;
    switch (which) {
    case PKV_WS_SCORE: return score_ws_bytes(shape);
    case PKV_WS_SEARCH: return kWsAlign;
    case PKV_WS_COMPACT:
        return round_up((size_t)shape->batch * shape->layers * shape->prompt_len * sizeof(int32_t),
                        kWsAlign);
    case PKV_WS_DECODE: return decode_ws_bytes(shape);
    default: return 0;
    }
}

extern "C" int prefixkv_score(const pkv_shape *shape, const void *q, pkv_strides qs, const void *k,
                              pkv_strides ks, const float *layer_scale, const float *lse,
                              float *scores, void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!shape_ok(shape) || !q || !k || !layer_scale || !scores) return PKV_ERR_INVALID_ARG;
    if (!shape_supported(shape)) return PKV_ERR_UNSUPPORTED;
    const int per16 = 16 / (int)esize(shape);
    int64_t st[8] = {qs.b, qs.l, qs.h, qs.n, ks.b, ks.l, ks.h, ks.n};
    for (int i = 0; i < 8; ++i)
        if (st[i] < 0 || st[i] % per16 != 0) return PKV_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k, 16)) return PKV_ERR_INVALID_ARG;
    if ((size_t)shape->batch * shape->layers > 65535 || shape->heads > 65535)
        return PKV_ERR_UNSUPPORTED;
    if (!ws || !aligned(ws, kWsAlign) || ws_bytes < score_ws_bytes(shape)) return PKV_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (shape->dtype == PKV_BF16) {
        if (score_tc_usable(shape, q, qs, k, ks)) {
            int rc = launch_score_tc(shape, q, qs, k, ks, layer_scale, lse, scores, ws, stream);
            if (rc >= 0) return rc;  // -1: layout not expressible as a tensor map, use the FMA path
        }
        if (shape->head_dim == 64)
            return launch_score_simt<__nv_bfloat16, 64>(shape, q, qs, k, ks, layer_scale, lse, scores,
                                                        ws, stream);
        return launch_score_simt<__nv_bfloat16, 128>(shape, q, qs, k, ks, layer_scale, lse, scores,
                                                     ws, stream);
    }
    if (shape->head_dim == 64)
        return launch_score_simt<float, 64>(shape, q, qs, k, ks, layer_scale, lse, scores, ws, stream);
    return launch_score_simt<float, 128>(shape, q, qs, k, ks, layer_scale, lse, scores, ws, stream);
}

extern "C" int prefixkv_gini(const pkv_shape *shape, const uint64_t *cum, double *gini,
                             void *cuda_stream)
{
    if (!shape_ok(shape) || !cum || !gini) return PKV_ERR_INVALID_ARG;
    gini_kernel<<<shape->batch * shape->layers, 256, 0, (cudaStream_t)cuda_stream>>>(
        cum, shape->prompt_len, gini);
    return check_launch("gini_kernel");
}

extern "C" int prefixkv_selftest_bounded_wait(int32_t which, int32_t *dev_status, void *cuda_stream)
{
    if (!dev_status) return PKV_ERR_INVALID_ARG;
    if (which == 0) return selftest_wait_score(dev_status, (cudaStream_t)cuda_stream);
    if (which == 1) return selftest_wait_stream(dev_status, (cudaStream_t)cuda_stream);
    return PKV_ERR_INVALID_ARG;
}

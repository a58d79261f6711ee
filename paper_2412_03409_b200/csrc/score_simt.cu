// Importance score (Sec. 3.2), FP32-FMA path: used for fp32 inputs, where the
// 1e-4 relative bar rules out reduced-precision tensor-core products.
//
//   pass 1: per query m, log2-sum-exp of the scaled causal logits (keys j <= m)
//   pass 2: per key n, sum over queries m >= n of exp2(logit - lse[m])
//   mean over heads in a fixed order (deterministic)
//
// The N x N probability matrix is never stored: both passes recompute 64 x 64
// logit tiles from Q and K staged through shared memory.
#include "common.cuh"

namespace pkv {

constexpr int TS = 64;   // tile side
constexpr int DC = 32;   // head-dim chunk staged per step
constexpr float kLog2eS = 1.4426950408889634f;

template <typename T>
__device__ __forceinline__ void stage_tile(const T *__restrict__ base, int64_t row_stride, int row0,
                                           int N, int d0, float (*dst)[DC + 1])
{
    for (int idx = threadIdx.x; idx < TS * DC; idx += 256) {
        int r = idx / DC, d = idx % DC;
        int row = row0 + r;
        dst[r][d] = row < N ? to_float(base[(int64_t)row * row_stride + d0 + d]) : 0.f;
    }
}

// Logits of one 64x64 tile: thread (ty, tx) holds rows ty + 16 i, cols tx + 16 j.
template <typename T, int D>
__device__ __forceinline__ void tile_logits(const T *__restrict__ qb, int64_t qsn, int m0,
                                            const T *__restrict__ kb, int64_t ksn, int n0, int N,
                                            float (*Qs)[DC + 1], float (*Ks)[DC + 1], int ty, int tx,
                                            float (&s)[4][4])
{
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
    for (int d0 = 0; d0 < D; d0 += DC) {
        __syncthreads();
        stage_tile<T>(qb, qsn, m0, N, d0, Qs);
        stage_tile<T>(kb, ksn, n0, N, d0, Ks);
        __syncthreads();
#pragma unroll 8
        for (int d = 0; d < DC; ++d) {
            float qv[4], kv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) qv[i] = Qs[ty + 16 * i][d];
#pragma unroll
            for (int j = 0; j < 4; ++j) kv[j] = Ks[tx + 16 * j][d];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) s[i][j] = fmaf(qv[i], kv[j], s[i][j]);
        }
    }
}

// grid (query tiles, H, B*L)
template <typename T, int D>
__global__ void __launch_bounds__(256)
score_lse_kernel(const T *__restrict__ q, pkv_strides qs, const T *__restrict__ k, pkv_strides ks,
                 const float *__restrict__ layer_scale, int L, int H, int N, float *__restrict__ lse2)
{
    __shared__ float Qs[TS][DC + 1], Ks[TS][DC + 1];
    const int mt = blockIdx.x, h = blockIdx.y, seg = blockIdx.z;
    const int b = seg / L, l = seg % L;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const T *qb = q + b * qs.b + l * qs.l + h * qs.h;
    const T *kb = k + b * ks.b + l * ks.l + h * ks.h;
    const float sc = layer_scale[l] * kLog2eS;
    float rmax[4], rsum[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { rmax[i] = -INFINITY; rsum[i] = 0.f; }
    for (int nt = 0; nt <= mt; ++nt) {
        float s[4][4];
        tile_logits<T, D>(qb, qs.n, mt * TS, kb, ks.n, nt * TS, N, Qs, Ks, ty, tx, s);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = mt * TS + ty + 16 * i;
            float tmax = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int n = nt * TS + tx + 16 * j;
                s[i][j] = (n <= m && n < N) ? s[i][j] * sc : -INFINITY;
                tmax = fmaxf(tmax, s[i][j]);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
            const float nm = fmaxf(rmax[i], tmax);
            float part = 0.f;
            if (nm > -INFINITY) {
#pragma unroll
                for (int j = 0; j < 4; ++j) part += exp2f(s[i][j] - nm);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
            rsum[i] = (nm > -INFINITY ? rsum[i] * exp2f(rmax[i] - nm) : 0.f) + part;
            rmax[i] = nm;
        }
    }
    if (tx == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = mt * TS + ty + 16 * i;
            if (m < N) lse2[((size_t)seg * H + h) * N + m] = rmax[i] + log2f(rsum[i]);
        }
    }
}

// grid (key tiles, H, B*L); lse_mul converts a caller-supplied natural-log lse.
template <typename T, int D>
__global__ void __launch_bounds__(256)
score_colsum_kernel(const T *__restrict__ q, pkv_strides qs, const T *__restrict__ k, pkv_strides ks,
                    const float *__restrict__ layer_scale, int L, int H, int N,
                    const float *__restrict__ lse, float lse_mul, float *__restrict__ partial)
{
    __shared__ float Qs[TS][DC + 1], Ks[TS][DC + 1];
    __shared__ float red[16][TS];
    const int nt = blockIdx.x, h = blockIdx.y, seg = blockIdx.z;
    const int b = seg / L, l = seg % L;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const T *qb = q + b * qs.b + l * qs.l + h * qs.h;
    const T *kb = k + b * ks.b + l * ks.l + h * ks.h;
    const float sc = layer_scale[l] * kLog2eS;
    const float *lrow = lse + ((size_t)seg * H + h) * N;
    const int ntiles = (N + TS - 1) / TS;
    float col[4] = {0.f, 0.f, 0.f, 0.f};
    for (int mt = nt; mt < ntiles; ++mt) {
        float s[4][4];
        tile_logits<T, D>(qb, qs.n, mt * TS, kb, ks.n, nt * TS, N, Qs, Ks, ty, tx, s);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = mt * TS + ty + 16 * i;
            const float lm = m < N ? lrow[m] * lse_mul : 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int n = nt * TS + tx + 16 * j;
                if (n <= m && m < N) col[j] += exp2f(fmaf(s[i][j], sc, -lm));
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) red[ty][tx + 16 * j] = col[j];
    __syncthreads();
    if (threadIdx.x < TS) {
        const int n = nt * TS + threadIdx.x;
        float t = 0.f;
#pragma unroll
        for (int r = 0; r < 16; ++r) t += red[r][threadIdx.x];
        if (n < N) partial[((size_t)seg * H + h) * N + n] = t;
    }
}

// scores[seg, n] = (1/H) * sum_h partial[seg, h, n], heads in index order.
// A set abort word (a bounded wait of the tensor-core passes ran out, so `partial` is not to be
// trusted) turns every score into NaN, which the selection stage reports as PKV_DEV_BAD_SCORE.
__global__ void head_mean_kernel(const float *__restrict__ partial, int H, int N, size_t total,
                                 float *__restrict__ scores, const int32_t *__restrict__ abort_word)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    dependent_entry();  // launched as a programmatic dependent of the pass that writes `partial`
    if (i >= total) return;
    if (abort_word && *abort_word != 0) {
        scores[i] = __int_as_float(0x7fc00000);
        return;
    }
    size_t seg = i / N;
    int n = (int)(i % N);
    float t = 0.f;
    for (int h = 0; h < H; ++h) t += partial[(seg * H + h) * N + n];
    scores[i] = t / (float)H;
}

int launch_head_mean(const float *partial, int H, int N, size_t total, float *scores, const int32_t *abort_word,
                     cudaStream_t st)
{
    cudaError_t e = launch_dependent(head_mean_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st,
                                     partial, H, N, total, scores, abort_word);
    if (e != cudaSuccess) {
        set_cuda_error(e, "head_mean_kernel");
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

template <typename T, int D>
int launch_score_simt(const pkv_shape *s, const void *q, pkv_strides qs, const void *k,
                      pkv_strides ks, const float *scale, const float *lse, float *scores,
                      void *ws, cudaStream_t st)
{
    const int B = s->batch, L = s->layers, H = s->heads, N = s->prompt_len;
    const size_t per = (size_t)B * L * H * N;
    float *partial = (float *)ws;
    float *lse2 = partial + per;
    const int tiles = (N + TS - 1) / TS;
    dim3 grid(tiles, H, B * L);
    float lse_mul = kLog2eS;
    if (!lse) {
        score_lse_kernel<T, D><<<grid, 256, 0, st>>>((const T *)q, qs, (const T *)k, ks, scale, L, H,
                                                     N, lse2);
        int rc = check_launch("score_lse_kernel");
        if (rc != PKV_OK) return rc;
        lse = lse2;
        lse_mul = 1.f;
    }
    score_colsum_kernel<T, D><<<grid, 256, 0, st>>>((const T *)q, qs, (const T *)k, ks, scale, L, H,
                                                    N, lse, lse_mul, partial);
    int rc = check_launch("score_colsum_kernel");
    if (rc != PKV_OK) return rc;
    return launch_head_mean(partial, H, N, (size_t)B * L * N, scores, nullptr, st);
}

#define PKV_INST(T, D)                                                                            \
    template int launch_score_simt<T, D>(const pkv_shape *, const void *, pkv_strides, const void *, \
                                         pkv_strides, const float *, const float *, float *, void *, \
                                         cudaStream_t);
PKV_INST(float, 64)
PKV_INST(float, 128)
PKV_INST(__nv_bfloat16, 64)
PKV_INST(__nv_bfloat16, 128)
#undef PKV_INST

}  // namespace pkv

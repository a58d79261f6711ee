// Exact budget and offline configuration (Sec. 3.3).  The paper says to "scale the resulting
// global prefix configuration to meet the target budget" after an inexact search, and to
// derive one configuration from a few sample prompts, without giving either formula.  Both
// are done here by one integer apportionment: every layer keeps its one mandatory row and
// the other budget - L rows are split in proportion to a weight per layer (largest remainder,
// ties to the lower layer, at most N rows per layer):
//   rescale:  weight[l] = len[b][l] - 1 of sample b's searched configuration
//   estimate: weight[l] = sum over the sample prompts of (len[k][l] - 1)
#include "common.cuh"

namespace pkv {

constexpr int kMaxLayers = 1024;

__device__ __forceinline__ int64_t block_sum_i64(int64_t v, int64_t *red)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    int64_t t = 0;
    for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += red[i];
    return t;
}

// One CTA per problem; thread l owns layer l.  `samples` rows of len_in are summed per problem.
__global__ void __launch_bounds__(kMaxLayers)
apportion_kernel(const int32_t *len_in, int samples, int L, int N, const int64_t *budget_dev,
                 int64_t budget_host, int32_t *len_out, int32_t *dev_status)
{
    __shared__ int64_t red[32];
    __shared__ int64_t s_fr[kMaxLayers];
    __shared__ int s_x[kMaxLayers], s_order[kMaxLayers];
    const int p = blockIdx.x, l = threadIdx.x;
    const bool mine = l < L;
    const int64_t budget = budget_dev ? budget_dev[p] : budget_host;
    int64_t w = 0;
    bool bad = false;
    if (mine) {
        for (int k = 0; k < samples; ++k) {
            int v = len_in[((size_t)p * samples + k) * L + l];
            if (v < 1 || v > N) {
                bad = true;
                v = v < 1 ? 1 : N;
            }
            w += v - 1;
        }
    }
    if (bad) raise_status(dev_status, p, PKV_DEV_BAD_LENGTH);
    if (budget < (int64_t)L) {  // uniform over the CTA
        if (l == 0) raise_status(dev_status, p, PKV_DEV_BUDGET_TOO_SMALL);
        if (mine) len_out[(size_t)p * L + l] = 1;
        return;
    }
    int64_t W = block_sum_i64(w, red);
    if (W == 0) {
        w = mine ? 1 : 0;
        W = L;
    }
    const int64_t extra = budget - L, cap = (int64_t)N - 1;
    const int64_t prod = w * extra;  // < 2^63: w <= 2^30 rows, extra <= 2^24 rows for supported sizes
    int64_t x = prod / W;
    const int64_t fr = prod % W;
    if (x > cap) x = cap;
    if (mine) {
        s_fr[l] = fr;
        s_x[l] = (int)x;
    }
    int64_t rem = extra - block_sum_i64(mine ? x : 0, red);
    // rank by (remainder descending, layer ascending)
    if (mine) {
        int rank = 0;
        for (int j = 0; j < L; ++j) rank += (s_fr[j] > fr) || (s_fr[j] == fr && j < l);
        s_order[rank] = l;
    }
    __syncthreads();
    if (l == 0) {
        while (rem > 0) {
            int given = 0;
            for (int i = 0; i < L && rem > 0; ++i) {
                const int ll = s_order[i];
                if (s_x[ll] < cap) {
                    ++s_x[ll];
                    --rem;
                    ++given;
                }
            }
            if (!given) break;  // every layer already keeps all N rows
        }
    }
    __syncthreads();
    if (mine) len_out[(size_t)p * L + l] = 1 + s_x[l];
}

static int threads_for(int L)
{
    int t = 32;
    while (t < L) t <<= 1;
    return t;
}

}  // namespace pkv

using namespace pkv;

extern "C" int prefixkv_rescale(const pkv_shape *shape, int32_t *len, const int64_t *budget_rows,
                                int32_t *dev_status, void *cuda_stream)
{
    if (!shape_ok(shape) || !len || !budget_rows || !dev_status) return PKV_ERR_INVALID_ARG;
    if (shape->layers > kMaxLayers) return PKV_ERR_UNSUPPORTED;
    apportion_kernel<<<shape->batch, threads_for(shape->layers), 0, (cudaStream_t)cuda_stream>>>(
        len, 1, shape->layers, shape->prompt_len, budget_rows, 0, len, dev_status);
    return check_launch("apportion_kernel");
}

extern "C" int prefixkv_estimate_config(const pkv_shape *shape, const int32_t *len, int64_t budget_rows,
                                        int32_t *len_out, int32_t *dev_status, void *cuda_stream)
{
    if (!shape_ok(shape) || !len || !len_out || !dev_status) return PKV_ERR_INVALID_ARG;
    if (shape->layers > kMaxLayers) return PKV_ERR_UNSUPPORTED;
    apportion_kernel<<<1, threads_for(shape->layers), 0, (cudaStream_t)cuda_stream>>>(
        len, shape->batch, shape->layers, shape->prompt_len, nullptr, budget_rows, len_out, dev_status);
    return check_launch("apportion_kernel");
}

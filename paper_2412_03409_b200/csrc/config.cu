// Exact budget and offline configuration (Sec. 3.3).  After the search the paper has the
// configuration scaled to the target budget, and it derives one configuration from a few sample
// prompts, without giving either formula.  Both are done here by one integer apportionment:
// every layer keeps its one mandatory row and the other budget - L rows are split in
// proportion to a weight per layer -- the floor of the quota first (at most N rows per layer),
// then what is left over one row at a time in the order of the division remainders (largest
// first, ties to the lower layer), round after round, to the layers that still have room:
//   rescale:  weight[l] = len[b][l] - 1 of sample b's searched configuration
//   estimate: weight[l] = sum over the sample prompts of (len[k][l] - 1)
// A configuration above its budget (a search ended by the threshold on the upper side) comes
// out shorter, never below one row per layer; one below it comes out longer.
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
// The left-over rows are dealt in whole rounds, all layers in parallel: while more rows are left
// than layers have room, every open layer takes min(rows left / open layers, its room) at once
// (what going round one row at a time would have given it by then); the last, partial round
// goes to the first `left` open layers in remainder order.
__global__ void __launch_bounds__(kMaxLayers)
apportion_kernel(const int32_t *len_in, int samples, int L, int N, const int64_t *budget_dev,
                 int64_t budget_host, int32_t *len_out, int32_t *dev_status)
{
    __shared__ int64_t red[32];
    __shared__ int64_t s_rem[kMaxLayers];
    __shared__ unsigned char s_open[kMaxLayers];  // by rank in remainder order: has the layer room?
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
    if (W == 0) {  // all weights zero: every layer counts the same
        w = mine ? 1 : 0;
        W = L;
    }
    const int64_t extra = budget - L, room0 = (int64_t)N - 1;
    const int64_t prod = w * extra;  // < 2^63: w <= 2^30 rows, extra <= 2^24 rows for supported sizes
    int64_t x = prod / W;
    const int64_t rem = prod % W;
    if (x > room0) x = room0;
    if (mine) s_rem[l] = rem;
    int64_t left = extra - block_sum_i64(mine ? x : 0, red);
    // this layer's place in the order (remainder descending, layer ascending)
    int rank = 0;
    if (mine)
        for (int j = 0; j < L; ++j) rank += (s_rem[j] > rem) || (s_rem[j] == rem && j < l);
    for (;;) {  // uniform over the CTA: `left` and the counts below are block-wide sums
        const int64_t room = mine ? room0 - x : 0;
        const int64_t open = block_sum_i64(room > 0 ? 1 : 0, red);
        if (left <= 0 || open == 0) break;
        if (left >= open) {
            // whole rounds: every open layer takes one row per round until it is full or the
            // rounds that all currently open layers can share are over
            const int64_t rounds = left / open;
            const int64_t take = room < rounds ? room : rounds;
            x += take;
            left -= block_sum_i64(take, red);
        } else {
            // the last round reaches only the first `left` open layers of the order
            if (mine) s_open[rank] = room > 0;
            __syncthreads();
            int ahead = 0;  // open layers before this one in the order
            if (mine && room > 0)
                for (int r = 0; r < rank; ++r) ahead += s_open[r];
            if (mine && room > 0 && ahead < left) x += 1;
            left = 0;
            break;
        }
    }
    if (mine) len_out[(size_t)p * L + l] = (int32_t)(1 + x);
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

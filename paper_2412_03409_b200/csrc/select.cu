// Selection stages: priority sequence + cumulative priority (Sec. 3.2) and the
// binary search for the global ratio p (Sec. 3.3, Eq. 1, Algorithm 1).
//
// All arithmetic that decides an index is integer: the sort key is the fp32 bit
// pattern (monotone for non-negative floats), cumulative sums are 2^-32 fixed
// point in uint64, and only p and the threshold p*total are fp64.
#include "common.cuh"

namespace pkv {

// ---------------------------------------------------------------------------
// One CTA per segment: sort (score desc, position asc) and inclusive scan.
// Keys are 64-bit (~score_bits << 32 | position) so that an ascending sort of
// unique keys yields the required order; a bitonic network in shared memory
// does the sort.  Padding keys are all ones and sort last.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint64_t weight_of_key(uint64_t key, bool &range_bad)
{
    uint32_t bits = ~(uint32_t)(key >> 32);
    if (bits > 0x7F7FFFFFu) return 0;  // padding, or a score already reported as bad
    double scaled = (double)__uint_as_float(bits) * 4294967296.0;  // exact
    if (scaled >= 9007199254740992.0) {
        range_bad = true;
        return 0;
    }
    return (uint64_t)__double2ll_rn(scaled);  // round half to even
}

__device__ __forceinline__ uint64_t add_check(uint64_t a, uint64_t b, bool &ovf)
{
    uint64_t s = a + b;
    ovf |= (s < a);
    return s;
}

__global__ void __launch_bounds__(1024)
sort_scan_kernel(const float *__restrict__ scores, int N, int P, int L, int32_t *__restrict__ order,
                 uint64_t *__restrict__ cum, int32_t *__restrict__ seg_flags)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t *keys = reinterpret_cast<uint64_t *>(smem_raw);  // [P]
    __shared__ uint64_t warp_tot[32];
    __shared__ int s_flags;

    const int seg = blockIdx.x;
    const int tid = threadIdx.x;
    const int nthr = blockDim.x;
    const float *src = scores + (size_t)seg * N;
    if (tid == 0) s_flags = 0;
    dependent_entry();  // set up while the kernel before it drained; its results are read from here on

    bool bad = false;
    for (int i = tid; i < P; i += nthr) {
        uint64_t key = ~0ull;
        if (i < N) {
            uint32_t bits = __float_as_uint(src[i]);
            if (bits == 0x80000000u) bits = 0;   // -0.0 is the same value as +0.0
            if (bits > 0x7F7FFFFFu) bad = true;  // negative, inf or NaN
            key = ((uint64_t)(~bits) << 32) | (uint32_t)i;
        }
        keys[i] = key;
    }
    __syncthreads();

    if (P == nthr) {
        // One key per thread, in a register: partners less than a warp apart exchange by shuffle,
        // the others through shared memory, two buffers in turn so that one barrier per such step
        // is enough.  (15 barriers instead of 55 for 1024 keys.)
        uint64_t key = keys[tid];
        uint64_t *buf[2] = {keys, keys + P};
        int cur = 1;  // keys[] itself was read above, before the barrier
        for (int k = 2; k <= P; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                uint64_t other;
                if (j >= 32) {
                    buf[cur][tid] = key;
                    __syncthreads();
                    other = buf[cur][tid ^ j];
                    cur ^= 1;
                } else {
                    other = __shfl_xor_sync(0xffffffffu, key, j);
                }
                const bool keep_min = ((tid & j) == 0) == ((tid & k) == 0);
                key = keep_min ? (key < other ? key : other) : (key > other ? key : other);
            }
        }
        __syncthreads();  // every read of keys[] / the buffers is over
        keys[tid] = key;
        __syncthreads();
    } else
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < (P >> 1); i += nthr) {
                int lo = ((i & ~(j - 1)) << 1) | (i & (j - 1));
                int hi = lo | j;
                bool up = (lo & k) == 0;
                uint64_t a = keys[lo], c = keys[hi];
                if ((a > c) == up) {
                    keys[lo] = c;
                    keys[hi] = a;
                }
            }
            __syncthreads();
        }
    }

    // Inclusive scan of the fixed-point weights, blocked over threads.
    const int ipt = P / nthr;  // P and nthr are powers of two, nthr <= P
    const int base = tid * ipt;
    bool range_bad = false, ovf = false;
    uint64_t local = 0;
    for (int i = 0; i < ipt; ++i)
        local = add_check(local, weight_of_key(keys[base + i], range_bad), ovf);
    uint64_t incl = local;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint64_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl = add_check(incl, up, ovf);
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        uint64_t t = (lane < (nthr >> 5)) ? warp_tot[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint64_t up = __shfl_up_sync(0xffffffffu, t, o);
            if (lane >= o) t = add_check(t, up, ovf);
        }
        warp_tot[lane] = t;  // inclusive over warps
    }
    __syncthreads();
    uint64_t run = add_check(incl - local, warp ? warp_tot[warp - 1] : 0, ovf);
    for (int i = 0; i < ipt; ++i) {
        int j = base + i;
        uint64_t key = keys[j];
        bool dummy = false;
        run = add_check(run, weight_of_key(key, dummy), ovf);
        if (j < N) {
            order[(size_t)seg * N + j] = (int32_t)(uint32_t)key;
            if (cum) cum[(size_t)seg * N + j] = run;
        }
    }
    if (tid == nthr - 1 && run >= (1ull << 53)) range_bad = true;
    if (bad) atomicOr(&s_flags, 1);
    if (range_bad || ovf) atomicOr(&s_flags, 2);
    __syncthreads();
    // What was found goes to the segment's slot of the length array (bit 0: a bad score, bit 1:
    // the fixed-point range); the kernel that follows turns the flags of a sample's layers into
    // its status word and then writes the lengths over them, so no separate clearing pass runs.
    if (tid == 0) seg_flags[seg] = s_flags;
}

// Status of a sample from the flags the sort kernel left in its layers' length slots.
__device__ __forceinline__ int status_from_flags(int flags)
{
    return (flags & 1) ? (int)PKV_DEV_BAD_SCORE : ((flags & 2) ? (int)PKV_DEV_RANGE : (int)PKV_DEV_OK);
}

// ---------------------------------------------------------------------------
// Length rule of Sec. 3.3 for one layer, evaluated by one warp: the number of
// cumulative values below theta, found by a 32-way search (every lane probes
// one pivot per round), plus one, clamped to [1, N].
// ---------------------------------------------------------------------------
// `pivot` is the lane's probe of the first round, c[(lane + 1) * chunk0 - 1] (or ~0 past the
// end): it does not depend on theta, so a caller that searches one row many times loads it once.
__device__ __forceinline__ int warp_length_for_theta(const uint64_t *__restrict__ c, int N,
                                                     uint64_t theta, int lane, uint64_t pivot)
{
    int a = 0, bnd = N;  // the count lies in [a, bnd]
    {
        const int chunk = (N + 31) >> 5;
        const int k = __popc(__ballot_sync(0xffffffffu, pivot < theta));
        a = k * chunk;
        const int nb = (k + 1) * chunk - 1;
        bnd = nb < N ? nb : N;
    }
    while (bnd > a) {
        int chunk = (bnd - a + 31) >> 5;
        int idx = a + (lane + 1) * chunk - 1;
        bool below = (idx < bnd) ? (c[idx] < theta) : false;
        int k = __popc(__ballot_sync(0xffffffffu, below));
        int na = a + k * chunk;
        int nb = a + (k + 1) * chunk - 1;
        a = na;
        bnd = nb < bnd ? nb : bnd;
    }
    int n = a + 1;
    return n > N ? N : (n < 1 ? 1 : n);
}

// One CTA per sample.  Warps take layers round-robin; every thread tracks the
// same (p1, p2) so control flow is uniform.  Two length buffers alternate so
// that one barrier per midpoint is enough.
__global__ void __launch_bounds__(1024)
search_kernel(const uint64_t *__restrict__ cum, const int64_t *__restrict__ budget_rows, int L,
              int N, double tol, int max_iters, int64_t slack, int64_t slack_over, int32_t *__restrict__ len,
              double *__restrict__ p_out, int32_t *__restrict__ iters_out, int32_t *dev_status)
{
    extern __shared__ int s_len[];  // [2][L]
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    const uint64_t *cb = cum + (size_t)b * L * N;
    dependent_entry();  // the sort kernel's sums and flags are complete
    const int64_t budget = budget_rows[b];
    {
        int flags = 0;
        for (int l = threadIdx.x; l < L; l += blockDim.x) flags |= len[(size_t)b * L + l];
        // (the block-wide "or" is of predicates, so one per bit)
        flags = (__syncthreads_or(flags & 1) ? 1 : 0) | (__syncthreads_or(flags & 2) ? 2 : 0);
        if (threadIdx.x == 0) dev_status[b] = status_from_flags(flags);  // overwrites: this call's status starts here
    }

    // What every midpoint needs of a layer's row and never changes: its total and this lane's
    // first-round probe.  Kept in registers for the first kHoist layers of the warp.
    constexpr int kHoist = 4;
    const int chunk0 = (N + 31) >> 5;
    double tot_r[kHoist];
    uint64_t piv_r[kHoist];
#pragma unroll
    for (int k = 0; k < kHoist; ++k) {
        const int l = warp + k * nwarp;
        tot_r[k] = 0.0;
        piv_r[k] = ~0ull;
        if (l < L) {
            const uint64_t *c = cb + (size_t)l * N;
            const int idx = (lane + 1) * chunk0 - 1;
            tot_r[k] = (double)c[N - 1];
            if (idx < N) piv_r[k] = c[idx];
        }
    }

    auto eval = [&](double p, int buf) -> int64_t {
        int *dst = s_len + buf * L;
#pragma unroll
        for (int k = 0; k < kHoist; ++k) {
            const int l = warp + k * nwarp;
            if (l < L) {
                int n = N;
                if (p < 1.0) {
                    const uint64_t theta = __double2ull_ru(__dmul_rn(p, tot_r[k]));
                    n = warp_length_for_theta(cb + (size_t)l * N, N, theta, lane, piv_r[k]);
                }
                if (lane == 0) dst[l] = n;
            }
        }
        for (int l = warp + kHoist * nwarp; l < L; l += nwarp) {
            const uint64_t *c = cb + (size_t)l * N;
            int n;
            if (p >= 1.0) {
                n = N;
            } else {
                const int idx = (lane + 1) * chunk0 - 1;
                double total = (double)c[N - 1];
                uint64_t theta = __double2ull_ru(__dmul_rn(p, total));
                n = warp_length_for_theta(c, N, theta, lane, idx < N ? c[idx] : ~0ull);
            }
            if (lane == 0) dst[l] = n;
        }
        __syncthreads();
        int64_t s = 0;
        for (int l = lane; l < L; l += 32) s += dst[l];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        return s;
    };

    double p_final = 0.0;
    int iters = 0, buf = 0;
    bool have = false;  // s_len[buf] already holds the lengths of p_final
    if (budget < (int64_t)L) {
        if (threadIdx.x == 0) raise_status(dev_status, b, PKV_DEV_BUDGET_TOO_SMALL);
    } else if ((int64_t)L * (int64_t)N <= budget) {
        p_final = 1.0;
    } else {
        double p1 = 0.0, p2 = 1.0;
        for (;;) {
            double p = (p1 + p2) * 0.5;
            if (p == p1 || p == p2 || iters == max_iters || p2 - p1 <= tol) {
                p_final = p1;
                break;
            }
            buf ^= 1;
            int64_t S = eval(p, buf);
            ++iters;
            int64_t delta = S - budget;
            if (delta >= -slack && delta <= slack_over) {  // within the threshold on delta (Sec. 3.3)
                p_final = p;
                have = true;
                break;
            }
            if (delta < 0) p1 = p; else p2 = p;
        }
    }
    if (!have) {
        buf ^= 1;
        eval(p_final, buf);
    }
    for (int l = threadIdx.x; l < L; l += blockDim.x) len[(size_t)b * L + l] = s_len[buf * L + l];
    if (threadIdx.x == 0) {
        p_out[b] = p_final;
        iters_out[b] = iters;
    }
}

// One CTA per sample: the caller's lengths, checked, and the sample's status word.
__global__ void __launch_bounds__(256)
take_lengths_kernel(const int32_t *__restrict__ len_in, int per_sample, int L, int N,
                    int32_t *__restrict__ len, int32_t *dev_status)
{
    const int b = blockIdx.x;
    dependent_entry();  // the sort kernel's flags are complete
    int flags = 0, bad = 0;
    for (int l = threadIdx.x; l < L; l += blockDim.x) {
        flags |= len[(size_t)b * L + l];
        int v = per_sample ? len_in[(size_t)b * L + l] : len_in[l];
        if (v < 1 || v > N) {
            bad = 1;
            v = v < 1 ? 1 : N;
        }
        len[(size_t)b * L + l] = v;
    }
    flags = (__syncthreads_or(flags & 1) ? 1 : 0) | (__syncthreads_or(flags & 2) ? 2 : 0);  // predicates: one per bit
    bad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
        const int st = status_from_flags(flags);
        dev_status[b] = st != PKV_DEV_OK ? st : (bad ? (int)PKV_DEV_BAD_LENGTH : (int)PKV_DEV_OK);
    }
}

static int launch_sort(const pkv_shape *s, const float *scores, int32_t *order, uint64_t *cum,
                       int32_t *seg_flags, cudaStream_t st)
{
    int N = s->prompt_len;
    int P = 32;
    while (P < N) P <<= 1;
    int nthr = P < 1024 ? P : 1024;
    size_t smem = (size_t)P * sizeof(uint64_t) * (P == nthr ? 2 : 1);  // one key per thread: two exchange buffers
    static bool attr_done[64] = {};
    if (smem > 48 * 1024) {
        int rc = ensure_dynamic_smem((const void *)sort_scan_kernel, 128 * 1024, attr_done);
        if (rc != PKV_OK) return rc;
    }
    cudaError_t e = launch_dependent(sort_scan_kernel, dim3(s->batch * s->layers), dim3(nthr), smem, st, scores, N, P,
                                     (int)s->layers, order, cum, seg_flags);
    if (e != cudaSuccess) {
        set_cuda_error(e, "sort_scan_kernel");
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

}  // namespace pkv

using namespace pkv;

extern "C" int prefixkv_search(const pkv_shape *shape, const float *scores,
                               const int64_t *budget_rows, double tol, int32_t max_iters,
                               int64_t slack_rows, int64_t slack_over_rows, int32_t *order, uint64_t *cum,
                               int32_t *len, double *p_out, int32_t *iters_out, int32_t *dev_status,
                               void *ws, size_t ws_bytes, void *cuda_stream)
{
    (void)ws; (void)ws_bytes;
    if (!shape_ok(shape) || !scores || !budget_rows || !order || !cum || !len || !p_out ||
        !iters_out || !dev_status || !(tol >= 0.0) || max_iters < 0 || slack_rows < 0 || slack_over_rows < 0)
        return PKV_ERR_INVALID_ARG;
    if (!shape_supported(shape)) return PKV_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int B = shape->batch, L = shape->layers, N = shape->prompt_len;
    if ((size_t)2 * L * sizeof(int) > 40 * 1024) return PKV_ERR_UNSUPPORTED;
    int rc = launch_sort(shape, scores, order, cum, len, st);
    if (rc != PKV_OK) return rc;
    cudaError_t e = launch_dependent(search_kernel, dim3(B), dim3(1024), 2 * L * sizeof(int), st,
                                     (const uint64_t *)cum, budget_rows, L, N, tol, (int)max_iters, slack_rows, slack_over_rows, len,
                                     p_out, iters_out, dev_status);
    if (e != cudaSuccess) {
        set_cuda_error(e, "search_kernel");
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

extern "C" int prefixkv_apply_lengths(const pkv_shape *shape, const float *scores,
                                      const int32_t *len_in, int32_t per_sample, int32_t *order,
                                      uint64_t *cum, int32_t *len, int32_t *dev_status, void *ws,
                                      size_t ws_bytes, void *cuda_stream)
{
    (void)ws; (void)ws_bytes;
    if (!shape_ok(shape) || !scores || !len_in || !order || !len || !dev_status)
        return PKV_ERR_INVALID_ARG;
    if (!shape_supported(shape)) return PKV_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int B = shape->batch, L = shape->layers, N = shape->prompt_len;
    if (len_in == len) return PKV_ERR_INVALID_ARG;  // (the output slots carry the sort's flags in between)
    int rc = launch_sort(shape, scores, order, cum, len, st);
    if (rc != PKV_OK) return rc;
    cudaError_t e = launch_dependent(take_lengths_kernel, dim3(B), dim3(256), 0, st, len_in, (int)per_sample, L, N, len,
                                     dev_status);
    if (e != cudaSuccess) {
        set_cuda_error(e, "take_lengths_kernel");
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

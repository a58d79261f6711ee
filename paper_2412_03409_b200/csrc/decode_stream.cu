// Streaming decode attention over the ragged cache (Sec. 3.1, Fig. 2a), the
// bandwidth-bound form of the decode step.
//
// Work is cut into units of up to four consecutive cache rows of one segment and
// the flat unit list is divided evenly over one persistent CTA per SM, so ragged
// per-layer lengths cost no imbalance.  A producer thread streams each unit's K
// rows and V rows (contiguous in the token-major cache) into a shared-memory ring
// with bulk asynchronous copies that complete on mbarriers; consumer warps own
// heads, keep q, the running softmax state and the output accumulator in
// registers, and read the ring with conflict-free 16-byte loads.  A CTA that
// covers only part of a segment leaves an un-normalised partial in scratch; the
// last CTA to arrive at the segment (a counter, no waiting) merges them.  The
// last CTA of the grid bumps the lengths, after every CTA has read them.
#include <cstdlib>

#include "common.cuh"

namespace pkv {

constexpr int kUnitRows = 4;
constexpr int kMaxActive = 2048;
constexpr int kMaxStages = 8;
constexpr int kDynSmemMax = 226 * 1024;  // 227 KiB per CTA less the kernel's static variables
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kLog2eD = 1.4426950408889634f;

struct DecodeArgs {
    const void *q, *k_new, *v_new;
    void *ck, *cv, *out;
    const int64_t *row_offset;
    int32_t *len;
    const int32_t *cap;
    int32_t *arrive;  // [B*L + 1], zero between calls
    const float *layer_scale;
    float *scratch;
    int32_t *dev_status;
    int L, H, layer_begin, nl, nact, nseg_total, nstages, nwarps;
    uint32_t row_bytes;
};

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_addr(dst)),
        "l"(src), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}
__device__ __forceinline__ void consumer_barrier(int nthreads)
{
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int VE = 4;
    __device__ static void unpack(const uint4 &r, float *x)
    {
        x[0] = __uint_as_float(r.x); x[1] = __uint_as_float(r.y);
        x[2] = __uint_as_float(r.z); x[3] = __uint_as_float(r.w);
    }
    __device__ static uint4 pack(const float *x)
    {
        return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]),
                          __float_as_uint(x[3]));
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int VE = 8;
    __device__ static void unpack(const uint4 &r, float *x)
    {
        x[0] = __uint_as_float(r.x << 16); x[1] = __uint_as_float(r.x & 0xffff0000u);
        x[2] = __uint_as_float(r.y << 16); x[3] = __uint_as_float(r.y & 0xffff0000u);
        x[4] = __uint_as_float(r.z << 16); x[5] = __uint_as_float(r.z & 0xffff0000u);
        x[6] = __uint_as_float(r.w << 16); x[7] = __uint_as_float(r.w & 0xffff0000u);
    }
    __device__ static uint4 pack(const float *x)
    {
        __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]), b = __floats2bfloat162_rn(x[2], x[3]);
        __nv_bfloat162 c = __floats2bfloat162_rn(x[4], x[5]), d = __floats2bfloat162_rn(x[6], x[7]);
        return make_uint4(*reinterpret_cast<uint32_t *>(&a), *reinterpret_cast<uint32_t *>(&b),
                          *reinterpret_cast<uint32_t *>(&c), *reinterpret_cast<uint32_t *>(&d));
    }
};

// Owner CTA of unit u when U units are spread over G CTAs as [floor(cU/G), floor((c+1)U/G)).
__device__ __forceinline__ int unit_owner(int u, int G, int U)
{
    return (int)((((int64_t)u + 1) * G - 1) / U);
}

// LPR lanes share one (row, head): lane c of a group holds 16-byte vectors c, c + LPR, ...
// HPW heads per consumer warp.  Block = nwarps consumer warps + 1 producer warp.
template <typename T, int D, int LPR, int HPW, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) decode_stream_kernel(const DecodeArgs a)
{
    constexpr int VE = Vec<T>::VE;
    constexpr int NV = D / VE / LPR;  // vectors per lane
    constexpr int EPL = NV * VE;      // elements per lane
    constexpr int GPW = 32 / LPR;     // row groups per warp
    static_assert(NV >= 1, "too many lanes per row");
    constexpr int kSlotStride = D + 4;  // acc[D], max, sum; padded so every head starts on 16 bytes

    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t slot_bytes = kUnitRows * a.row_bytes;
    unsigned char *ring = smem;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + (size_t)a.nstages * slot_bytes);
    uint64_t *empty = full + kMaxStages;
    int *P = reinterpret_cast<int *>(empty + kMaxStages);  // [nact + 1] unit prefix
    int *nlen = P + a.nact + 1;                            // [nact] rows, or -1 when not active
    __shared__ int s_flag, s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NW = a.nwarps;
    const int H = a.H;

    // ---- plan: units per active segment, exclusive scan (warp 0) -------------------------
    if (tid == 0) {
        s_abort = 0;
        for (int i = 0; i < a.nstages; ++i) {
            mbar_init(full + i, 1);
            mbar_init(empty + i, NW);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        int run = 0;
        for (int base = 0; base < a.nact; base += 32) {
            int si = base + lane, units = 0, n = -1;
            if (si < a.nact) {
                int seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
                int ln = a.len[seg], cp = a.cap[seg];
                if (ln >= 1 && ln < cp) {
                    n = ln;
                    units = (ln + kUnitRows - 1) / kUnitRows;
                }
                nlen[si] = n;
            }
            int incl = units;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            if (si < a.nact) P[si] = run + incl - units;
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) P[a.nact] = run;
    }
    __syncthreads();
    const int U = P[a.nact];
    const int G = (int)gridDim.x < U ? (int)gridDim.x : U;  // CTAs that get work
    const int cta = blockIdx.x;

    // segments that cannot take another row: report, write zeros
    for (int si = cta; si < a.nact; si += gridDim.x) {
        if (nlen[si] >= 0) continue;
        const int b = si / a.nl, seg = b * a.L + a.layer_begin + si % a.nl;
        if (tid == 0) raise_status(a.dev_status, b, PKV_DEV_CAPACITY);
        T *o = reinterpret_cast<T *>(a.out) + (size_t)seg * H * D;
        for (int e = tid; e < H * D; e += blockDim.x) o[e] = from_float<T>(0.f);
    }

    int u0 = 0, u1 = 0;
    if (cta < G) {
        u0 = (int)((int64_t)cta * U / G);
        u1 = (int)((int64_t)(cta + 1) * U / G);
    }

    if (warp == NW) {
        // ---- producer ---------------------------------------------------------------------
        if (lane == 0 && u0 < u1) {
            int si = 0, it = 0;
            // binary search for the segment of u0
            {
                int lo = 0, hi = a.nact;
                while (hi - lo > 1) {
                    int mid = (lo + hi) >> 1;
                    if (P[mid] <= u0) lo = mid; else hi = mid;
                }
                si = lo;
            }
            bool ok = true;
            for (int u = u0; u < u1 && ok; ++u) {
                while (u >= P[si + 1]) ++si;
                const int seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
                const int r0 = (u - P[si]) * kUnitRows;
                const int cnt = min(kUnitRows, nlen[si] - r0);
                const uint32_t bytes = (uint32_t)cnt * a.row_bytes;
                const size_t src_off = (size_t)(a.row_offset[seg] + r0) * a.row_bytes;
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {
                    const int slot = it % a.nstages;
                    const uint32_t ph = (uint32_t)(it / a.nstages) & 1u;
                    if (!mbar_wait(empty + slot, ph ^ 1u) || *(volatile int *)&s_abort) {
                        atomicExch(&s_abort, 1);
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(full + slot, bytes);
                    const unsigned char *src =
                        reinterpret_cast<const unsigned char *>(kv ? a.cv : a.ck) + src_off;
                    bulk_load(ring + (size_t)slot * slot_bytes, src, bytes, full + slot);
                    ++it;
                }
            }
            if (!ok) {
                // let copies already issued land before the CTA can exit
                for (int j = 0; j < it; ++j)
                    if (it - j <= a.nstages) mbar_wait(full + j % a.nstages, (uint32_t)(j / a.nstages) & 1u);
            }
        }
    } else if (u0 < u1) {
        // ---- consumers --------------------------------------------------------------------
        const int g = lane / LPR, c = lane % LPR;
        const int h0 = warp * HPW;
        float qf[HPW][EPL], acc[HPW][EPL], m[HPW], l[HPW], s[HPW][kUnitRows / GPW];
        int si = 0, it = 0;
        {
            int lo = 0, hi = a.nact;
            while (hi - lo > 1) {
                int mid = (lo + hi) >> 1;
                if (P[mid] <= u0) lo = mid; else hi = mid;
            }
            si = lo;
        }
        bool fresh = true;  // state must be reset and q loaded for segment si
        bool timed_out = false;
        for (int u = u0; u < u1; ++u) {
            if (u >= P[si + 1]) {
                while (u >= P[si + 1]) ++si;
                fresh = true;
            }
            const int b = si / a.nl, lyr = a.layer_begin + si % a.nl;
            const int seg = b * a.L + lyr;
            const int n = nlen[si];
            const size_t seg_vec = (size_t)seg * H * D;
            if (fresh) {
                fresh = false;
                const float sc = a.layer_scale[lyr] * kLog2eD;
#pragma unroll
                for (int hh = 0; hh < HPW; ++hh) {
                    m[hh] = -INFINITY;
                    l[hh] = 0.f;
                    const int h = h0 + hh;
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        float x[VE];
                        if (h < H) {
                            const uint4 raw = __ldg(reinterpret_cast<const uint4 *>(
                                reinterpret_cast<const T *>(a.q) + seg_vec + (size_t)h * D +
                                (v * LPR + c) * VE));
                            Vec<T>::unpack(raw, x);
                        }
#pragma unroll
                        for (int i = 0; i < VE; ++i) {
                            qf[hh][v * VE + i] = h < H ? x[i] * sc : 0.f;
                            acc[hh][v * VE + i] = 0.f;
                        }
                    }
                }
            }
            const int r0 = (u - P[si]) * kUnitRows;
            const int cnt = min(kUnitRows, n - r0);

            // ---- K item: logits of up to four rows --------------------------------------
            {
                const int slot = it % a.nstages;
                const uint32_t ph = (uint32_t)(it / a.nstages) & 1u;
                if (!timed_out && !*(volatile int *)&s_abort && !mbar_wait(full + slot, ph)) {
                    timed_out = true;
                    atomicExch(&s_abort, 1);
                }
                const unsigned char *kb = ring + (size_t)slot * slot_bytes;
#pragma unroll
                for (int j = 0; j < kUnitRows / GPW; ++j) {
                    const int rr = g + j * GPW;
#pragma unroll
                    for (int hh = 0; hh < HPW; ++hh) {
                        const int h = h0 + hh;
                        float dot = 0.f;
                        if (rr < cnt && h < H) {
                            const unsigned char *row = kb + (size_t)rr * a.row_bytes + (size_t)h * D * sizeof(T);
#pragma unroll
                            for (int v = 0; v < NV; ++v) {
                                const uint4 raw = *reinterpret_cast<const uint4 *>(row + (v * LPR + c) * 16);
                                float x[VE];
                                Vec<T>::unpack(raw, x);
#pragma unroll
                                for (int i = 0; i < VE; ++i) dot = fmaf(qf[hh][v * VE + i], x[i], dot);
                            }
                        }
#pragma unroll
                        for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                        s[hh][j] = dot;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty + slot);
                ++it;
            }
            // ---- V item: softmax update and accumulation ----------------------------------
            {
                const int slot = it % a.nstages;
                const uint32_t ph = (uint32_t)(it / a.nstages) & 1u;
                if (!timed_out && !*(volatile int *)&s_abort && !mbar_wait(full + slot, ph)) {
                    timed_out = true;
                    atomicExch(&s_abort, 1);
                }
                const unsigned char *vb = ring + (size_t)slot * slot_bytes;
#pragma unroll
                for (int j = 0; j < kUnitRows / GPW; ++j) {
                    const int rr = g + j * GPW;
#pragma unroll
                    for (int hh = 0; hh < HPW; ++hh) {
                        const int h = h0 + hh;
                        if (rr < cnt && h < H) {
                            const float sv = s[hh][j];
                            if (sv > m[hh]) {
                                const float corr = exp2f(m[hh] - sv);
                                l[hh] *= corr;
#pragma unroll
                                for (int i = 0; i < EPL; ++i) acc[hh][i] *= corr;
                                m[hh] = sv;
                            }
                            const float p = exp2f(sv - m[hh]);
                            l[hh] += p;
                            const unsigned char *row = vb + (size_t)rr * a.row_bytes + (size_t)h * D * sizeof(T);
#pragma unroll
                            for (int v = 0; v < NV; ++v) {
                                const uint4 raw = *reinterpret_cast<const uint4 *>(row + (v * LPR + c) * 16);
                                float x[VE];
                                Vec<T>::unpack(raw, x);
#pragma unroll
                                for (int i = 0; i < VE; ++i)
                                    acc[hh][v * VE + i] = fmaf(p, x[i], acc[hh][v * VE + i]);
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty + slot);
                ++it;
            }

            const bool seg_end = (u == P[si + 1] - 1);
            if (seg_end) {
                // ---- the row appended this step: taken from the inputs, stored as row n -------
                const size_t row_vec = (size_t)(a.row_offset[seg] + n) * H * D;
#pragma unroll
                for (int hh = 0; hh < HPW; ++hh) {
                    const int h = h0 + hh;
                    float dot = 0.f;
                    uint4 vraw[NV];
                    if (h < H) {
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            const size_t e = seg_vec + (size_t)h * D + (v * LPR + c) * VE;
                            const uint4 kraw = __ldg(reinterpret_cast<const uint4 *>(
                                reinterpret_cast<const T *>(a.k_new) + e));
                            vraw[v] = __ldg(reinterpret_cast<const uint4 *>(
                                reinterpret_cast<const T *>(a.v_new) + e));
                            if (g == 0) {
                                const size_t d = row_vec + (size_t)h * D + (v * LPR + c) * VE;
                                *reinterpret_cast<uint4 *>(reinterpret_cast<T *>(a.ck) + d) = kraw;
                                *reinterpret_cast<uint4 *>(reinterpret_cast<T *>(a.cv) + d) = vraw[v];
                            }
                            float x[VE];
                            Vec<T>::unpack(kraw, x);
#pragma unroll
                            for (int i = 0; i < VE; ++i) dot = fmaf(qf[hh][v * VE + i], x[i], dot);
                        }
                    }
#pragma unroll
                    for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                    if (g == 0 && h < H) {
                        if (dot > m[hh]) {
                            const float corr = exp2f(m[hh] - dot);
                            l[hh] *= corr;
#pragma unroll
                            for (int i = 0; i < EPL; ++i) acc[hh][i] *= corr;
                            m[hh] = dot;
                        }
                        const float p = exp2f(dot - m[hh]);
                        l[hh] += p;
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            float x[VE];
                            Vec<T>::unpack(vraw[v], x);
#pragma unroll
                            for (int i = 0; i < VE; ++i)
                                acc[hh][v * VE + i] = fmaf(p, x[i], acc[hh][v * VE + i]);
                        }
                    }
                }
            }
            if (seg_end || u == u1 - 1) {
                // ---- close this CTA's piece of the segment ---------------------------------------
                const int c_first = unit_owner(P[si], G, U), c_last = unit_owner(P[si + 1] - 1, G, U);
                const int ncontrib = c_last - c_first + 1;
#pragma unroll
                for (int hh = 0; hh < HPW; ++hh) {
                    // merge the row groups of the warp
                    float M = m[hh];
#pragma unroll
                    for (int o = LPR; o < 32; o <<= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
                    const float f = m[hh] == -INFINITY ? 0.f : exp2f(m[hh] - M);
                    float lt = l[hh] * f;
#pragma unroll
                    for (int o = LPR; o < 32; o <<= 1) lt += __shfl_xor_sync(0xffffffffu, lt, o);
#pragma unroll
                    for (int i = 0; i < EPL; ++i) {
                        float t = acc[hh][i] * f;
#pragma unroll
                        for (int o = LPR; o < 32; o <<= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                        acc[hh][i] = t;
                    }
                    const int h = h0 + hh;
                    if (g == 0 && h < H) {
                        if (ncontrib == 1) {
                            const float inv = 1.f / lt;
#pragma unroll
                            for (int v = 0; v < NV; ++v) {
                                float x[VE];
#pragma unroll
                                for (int i = 0; i < VE; ++i) x[i] = acc[hh][v * VE + i] * inv;
                                *reinterpret_cast<uint4 *>(reinterpret_cast<T *>(a.out) + seg_vec +
                                                           (size_t)h * D + (v * LPR + c) * VE) = Vec<T>::pack(x);
                            }
                        } else {
                            float *slot = a.scratch + ((size_t)(cta + si) * H + h) * kSlotStride;
#pragma unroll
                            for (int v = 0; v < NV; ++v)
#pragma unroll
                                for (int i = 0; i < VE; i += 4)
                                    *reinterpret_cast<float4 *>(slot + (v * LPR + c) * VE + i) =
                                        make_float4(acc[hh][v * VE + i], acc[hh][v * VE + i + 1],
                                                    acc[hh][v * VE + i + 2], acc[hh][v * VE + i + 3]);
                            if (c == 0) {
                                slot[D] = M;
                                slot[D + 1] = lt;
                            }
                        }
                    }
                }
                if (ncontrib > 1) {
                    __threadfence();
                    consumer_barrier(NW * 32);
                    if (tid == 0) {
                        __threadfence();
                        const int old = atomicAdd(a.arrive + seg, 1);
                        s_flag = (old == ncontrib - 1);
                    }
                    consumer_barrier(NW * 32);
                    if (s_flag) {
                        __threadfence();
                        for (int hh = 0; hh < HPW; ++hh) {
                            const int h = h0 + hh;
                            if (h >= H) continue;
                            float M = -INFINITY;
                            for (int cc = c_first; cc <= c_last; ++cc)
                                M = fmaxf(M, __ldcg(a.scratch + ((size_t)(cc + si) * H + h) * kSlotStride + D));
                            float z = 0.f, o[D / 32];
#pragma unroll
                            for (int i = 0; i < D / 32; ++i) o[i] = 0.f;
                            for (int cc = c_first; cc <= c_last; ++cc) {
                                const float *slot = a.scratch + ((size_t)(cc + si) * H + h) * kSlotStride;
                                const float w = exp2f(__ldcg(slot + D) - M);
                                z += w * __ldcg(slot + D + 1);
#pragma unroll
                                for (int i = 0; i < D / 32; ++i) o[i] += w * __ldcg(slot + lane + 32 * i);
                            }
                            const float inv = 1.f / z;
                            T *dst = reinterpret_cast<T *>(a.out) + seg_vec + (size_t)h * D;
#pragma unroll
                            for (int i = 0; i < D / 32; ++i) dst[lane + 32 * i] = from_float<T>(o[i] * inv);
                        }
                        consumer_barrier(NW * 32);
                        if (tid == 0) a.arrive[seg] = 0;
                    }
                }
                fresh = true;
            }
        }
        if (timed_out && lane == 0) raise_status(a.dev_status, 0, PKV_DEV_TIMEOUT);
    }

    // ---- last CTA of the grid: every CTA has read the lengths, so they can grow ----------
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const int old = atomicAdd(a.arrive + a.nseg_total, 1);
        s_flag = (old == (int)gridDim.x - 1);
    }
    __syncthreads();
    if (s_flag) {
        for (int si = tid; si < a.nact; si += blockDim.x) {
            if (nlen[si] < 0) continue;
            const int seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
            a.len[seg] = nlen[si] + 1;
        }
        if (tid == 0) a.arrive[a.nseg_total] = 0;
    }
}

size_t decode_stream_ws_bytes(const pkv_shape *s)
{
    size_t slots = 256 + (size_t)s->batch * s->layers;
    return round_up(slots * s->heads * (s->head_dim + 4) * sizeof(float), kWsAlign);
}

template <typename T, int D, int LPR, int HPW, int MAXT>
static int launch_variant(const DecodeArgs &a, int sms, cudaStream_t st)
{
    static bool done[64] = {};
    const size_t slot_bytes = (size_t)kUnitRows * a.row_bytes;
    const size_t smem = (size_t)a.nstages * slot_bytes + 2 * kMaxStages * sizeof(uint64_t) +
                        (size_t)(2 * a.nact + 1) * sizeof(int) + 16;
    if ((a.nwarps + 1) * 32 > MAXT) return -1;
    int rc = ensure_dynamic_smem((const void *)decode_stream_kernel<T, D, LPR, HPW, MAXT>, kDynSmemMax, done);
    if (rc != PKV_OK) return rc;
    decode_stream_kernel<T, D, LPR, HPW, MAXT><<<sms, (a.nwarps + 1) * 32, smem, st>>>(a);
    return check_launch("decode_stream_kernel");
}

// Returns PKV_OK, an error, or -1 when this shape is outside what the streaming kernel covers.
int launch_decode_stream(const pkv_shape *s, pkv_cache *c, const void *q, const void *kn,
                         const void *vn, const float *scale, int lb, int le, void *out,
                         int32_t *dev_status, void *ws, cudaStream_t st)
{
    if (!c->arrive) return -1;
    const int H = s->heads, D = s->head_dim, nl = le - lb, nact = s->batch * nl;
    if (nact > kMaxActive || H > 64) return -1;
    const size_t es = esize(s);
    const uint32_t row_bytes = (uint32_t)((size_t)H * D * es);
    const size_t slot_bytes = (size_t)kUnitRows * row_bytes;
    const size_t meta = 2 * kMaxStages * sizeof(uint64_t) + (size_t)(2 * nact + 1) * sizeof(int) + 256;
    const size_t budget = kDynSmemMax - meta;
    int nstages = (int)(budget / slot_bytes);
    if (nstages > kMaxStages) nstages = kMaxStages;
    if (nstages < 3) return -1;

    static int sm_count[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    int sms = (dev >= 0 && dev < 64) ? sm_count[dev] : 0;
    if (!sms) {
        cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) {
            set_cuda_error(e, "cudaDeviceGetAttribute(sm count)");
            return PKV_ERR_CUDA;
        }
        if (dev >= 0 && dev < 64) sm_count[dev] = sms;
    }
    if (sms > 256) sms = 256;

    DecodeArgs a;
    a.q = q; a.k_new = kn; a.v_new = vn; a.ck = c->k; a.cv = c->v; a.out = out;
    a.row_offset = c->row_offset; a.len = c->len; a.cap = c->cap; a.arrive = c->arrive;
    a.layer_scale = scale; a.scratch = (float *)ws; a.dev_status = dev_status;
    a.L = s->layers; a.H = H; a.layer_begin = lb; a.nl = nl; a.nact = nact;
    a.nseg_total = s->batch * s->layers; a.nstages = nstages; a.row_bytes = row_bytes;

    const bool bf = s->dtype == PKV_BF16;
    const int vec_per_head = D / (int)(16 / es);
    // (lanes per row, heads per warp): fewer, fatter warps once H > 16 so that the register
    // file of each SM sub-partition holds the per-head state without spilling.
    int lpr = 8, hpw = H <= 16 ? 1 : 4;
    if (H > 32 && vec_per_head >= 16) lpr = 16;
    if (const char *env = getenv("PKV_DECODE_VARIANT")) {
        int code = atoi(env);
        if (code > 0) { lpr = code / 10; hpw = code % 10; }
    }
    if (vec_per_head < lpr) return -1;
    a.nwarps = (H + hpw - 1) / hpw;
#define PKV_V(T, DD, LPR, HPW, MAXT) \
    if (lpr == LPR && hpw == HPW && (a.nwarps + 1) * 32 <= MAXT) \
        return launch_variant<T, DD, LPR, HPW, MAXT>(a, sms, st)
#define PKV_FAMILY(T, DD)            \
    PKV_V(T, DD, 8, 1, 544);         \
    PKV_V(T, DD, 8, 2, 544);         \
    PKV_V(T, DD, 8, 4, 288);         \
    PKV_V(T, DD, 8, 4, 544)
    if (bf && D == 128) {
        PKV_FAMILY(__nv_bfloat16, 128);
        PKV_V(__nv_bfloat16, 128, 16, 2, 544);
        PKV_V(__nv_bfloat16, 128, 16, 4, 288);
        PKV_V(__nv_bfloat16, 128, 16, 4, 544);
    } else if (bf && D == 64) {
        PKV_FAMILY(__nv_bfloat16, 64);
    } else if (!bf && D == 128) {
        PKV_FAMILY(float, 128);
        PKV_V(float, 128, 16, 2, 544);
        PKV_V(float, 128, 16, 4, 288);
        PKV_V(float, 128, 16, 4, 544);
    } else if (!bf && D == 64) {
        PKV_FAMILY(float, 64);
        PKV_V(float, 64, 16, 4, 544);
    }
#undef PKV_FAMILY
#undef PKV_V
    return -1;
}

}  // namespace pkv

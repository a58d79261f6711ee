// Streaming decode attention over the ragged cache (Sec. 3.1, Fig. 2a), the
// bandwidth-bound form of the decode step.
//
// Work is cut into units of up to UR consecutive rows of one segment (the row
// being appended counts as the segment's last row) and the flat unit list is
// divided evenly over one persistent CTA per SM, so ragged per-layer lengths cost
// no imbalance.  One producer thread moves everything the CTA reads -- q, each
// unit's K rows and V rows (contiguous in the token-major cache) and the new
// k/v row -- into shared memory with bulk asynchronous copies that complete on
// mbarriers; no other thread loads from global memory while the stream runs, so
// nothing queues behind the bulk traffic.  Consumer warps own heads, keep q, the
// running softmax state and the output accumulator in registers, and read the
// ring with conflict-free 16-byte loads.  A CTA that covers a whole segment
// writes its output directly; one that covers part of it leaves an
// un-normalised partial in scratch.  A small second kernel, launched as a
// programmatic dependent so that its launch overlaps the stream, merges the
// partials of split segments in parallel over all SMs and writes the lengths.
// (Merging inside the stream kernel instead, by the last CTA to arrive at a
// counter, was measured slower: its fence, counter and loads wait behind the
// other CTAs' bulk traffic, while the second kernel finds the memory system idle.)
#include "common.cuh"

namespace pkv {

constexpr int kMaxActive = 1024;
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
    const float *layer_scale;
    float *scratch;   // partial slots
    int *plan;        // [nact] int4 records written by the stream kernel for the merge kernel
    int32_t *dev_status;
    const int32_t *len0;  // [B*L] rows kept by compaction        } only with
    int32_t *gen;         // [B*L] tokens decoded so far          } decode-time
    int32_t *slot_ring;   // [B*L][distance + 1] rows of recent tokens } pruning
    int evict_distance, N;
    int L, H, layer_begin, nl, nact, nseg_total, nstages, nwarps;
    uint32_t row_bytes;
    int64_t total_cap_rows;
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
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, uint32_t limit = kSpinLimit)
{
    for (uint32_t i = 0; i < limit; ++i)
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

// U units over G CTAs (G <= U): the first U % G CTAs take U / G + 1 units, the rest U / G.
__device__ __forceinline__ int first_unit(int c, int q, int rem) { return c * q + min(c, rem); }
__device__ __forceinline__ int unit_owner(int u, int q, int rem)
{
    const int big = rem * (q + 1);
    return u < big ? u / (q + 1) : rem + (u - big) / q;
}

// Wait for a barrier phase; `dead` latches once a bounded wait has run out anywhere in
// the CTA, after which nothing waits any more (the results are then unspecified).
__device__ __forceinline__ void wait_phase(uint64_t *bar, uint32_t parity, bool &dead, int *abort_flag,
                                           uint32_t limit = kSpinLimit)
{
    if (dead || mbar_try_wait(bar, parity)) return;
    if (*(volatile int *)abort_flag || !mbar_wait(bar, parity, limit)) {
        dead = true;
        atomicExch(abort_flag, 1);
    }
}

// One warp waits, with a short limit, on a barrier phase that nothing completes: the give-up path
// of the streaming kernel in isolation.
__global__ void selftest_wait_stream_kernel(int32_t *dev_status, uint32_t limit)
{
    __shared__ uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool dead = false;
    if (threadIdx.x == 0) wait_phase(&bar, 0u, dead, &s_abort, limit);
    __syncthreads();
    wait_phase(&bar, 0u, dead, &s_abort, limit);  // the other lanes see the flag and stop at once
    if (threadIdx.x == 0 && dead && s_abort) raise_status(dev_status, 0, PKV_DEV_TIMEOUT);
}

int selftest_wait_stream(int32_t *dev_status, cudaStream_t st)
{
    selftest_wait_stream_kernel<<<1, 32, 0, st>>>(dev_status, 4096u);
    return check_launch("selftest_wait_stream_kernel");
}

// What this step does to active segment si: the rows it attends over (the new row included),
// or -1 when the segment cannot take the row (full, never compacted, or outside the cache);
// the row the new token is written to; the length afterwards.  Without decode-time pruning
// the new row is appended.  With it (Sec. 3.1: prune at a fixed distance to the latest token,
// keep the layer's proportion): when generated token g would push the layer past
// floor(len0 * (N + g + 1) / N) rows and token g - distance is still cached, the new row
// takes that token's slot instead and the length stays.
struct SegPlan {
    int rows, dst, len_after;
    bool evict;
    int64_t off;
};
__device__ __forceinline__ SegPlan segment_plan(const DecodeArgs &a, int si)
{
    const int seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
    const int ln = a.len[seg], cp = a.cap[seg];
    SegPlan p;
    p.off = a.row_offset[seg];
    p.evict = false;
    p.dst = ln;
    bool ok = ln >= 1 && p.off >= 0 && p.off + cp <= a.total_cap_rows && ln <= cp;
    if (!a.k_new) {  // nothing to append: attend over the rows that are there
        p.dst = 0x3fffffff;
        p.rows = ok ? ln : -1;
        p.len_after = p.rows;
        return p;
    }
    const int d = a.evict_distance;
    if (ok && d > 0) {
        const int g = a.gen[seg];
        const int64_t target = ((int64_t)a.len0[seg] * ((int64_t)a.N + g + 1)) / a.N;
        if ((int64_t)ln + 1 > target && g >= d) {
            const int r = a.slot_ring[(size_t)seg * (d + 1) + (g - d) % (d + 1)];
            if (r >= 0 && r < ln) {
                p.evict = true;
                p.dst = r;
            }
        }
    }
    if (!p.evict && ln >= cp) ok = false;  // appending needs head-room
    p.rows = ok ? (p.evict ? ln : ln + 1) : -1;
    p.len_after = p.rows;
    return p;
}

struct Ring {
    int slot, nstages;
    uint32_t phase;
    __device__ __forceinline__ void advance()
    {
        if (++slot == nstages) {
            slot = 0;
            phase ^= 1u;
        }
    }
};

// LPR lanes share one (row, head): lane c of a group holds 16-byte vectors c, c + LPR, ...
// HPW heads per consumer warp, UR rows per unit.  Block = nwarps consumer warps + 1 producer warp.
template <typename T, int D, int LPR, int HPW, int UR, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) decode_stream_kernel(const DecodeArgs a)
{
    constexpr int VE = Vec<T>::VE;
    constexpr int NV = D / VE / LPR;  // vectors per lane
    constexpr int EPL = NV * VE;      // elements per lane
    constexpr int GPW = 32 / LPR;     // row groups per warp
    constexpr int RPG = UR / GPW;     // rows per group per unit
    constexpr int kSlotStride = D + 4;  // acc[D], max, sum; padded so every head starts on 16 bytes
    static_assert(NV >= 1 && RPG >= 1, "bad lane mapping");

    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t rb = a.row_bytes;
    const uint32_t slot_bytes = UR * rb;
    unsigned char *ring = smem;
    unsigned char *qbuf = ring + (size_t)a.nstages * slot_bytes;  // [2][rb]
    uint64_t *full = reinterpret_cast<uint64_t *>(qbuf + 2 * (size_t)rb);
    uint64_t *empty = full + kMaxStages;
    uint64_t *qfull = empty + kMaxStages;  // [2]
    uint64_t *qempty = qfull + 2;          // [2]
    int64_t *seg_off = reinterpret_cast<int64_t *>(qempty + 2);  // [nact] first row of the segment
    int *P = reinterpret_cast<int *>(seg_off + a.nact);          // [nact + 1] unit prefix
    int *seg_rows = P + a.nact + 1;                              // [nact] rows attended (new one included), or -1
    int *seg_dst = seg_rows + a.nact;                            // [nact] row the new token is written to
    __shared__ int s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NW = a.nwarps;
    const int H = a.H;

    // ---- plan: rows, first row and unit count of every active segment ---------------------
    if (tid == 0) {
        s_abort = 0;
        for (int i = 0; i < a.nstages; ++i) {
            mbar_init(full + i, 1);
            mbar_init(empty + i, NW);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(qfull + i, 1);
            mbar_init(qempty + i, NW);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        P[0] = 0;
    }
    // Launched as a programmatic dependent of whatever precedes it in the stream: everything
    // above overlapped that kernel's tail; its writes (lengths, cache rows) are visible from here.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int si = tid; si < a.nact; si += blockDim.x) {
        const SegPlan sp = segment_plan(a, si);
        seg_rows[si] = sp.rows;
        seg_dst[si] = sp.dst | (sp.evict ? (1 << 30) : 0);
        seg_off[si] = sp.off;
        P[si + 1] = sp.rows > 0 ? (sp.rows + UR - 1) / UR : 0;
    }
    __syncthreads();
    if (warp == 0) {
        int run = 0;
        for (int base = 0; base < a.nact; base += 32) {
            const int i = base + lane;
            int incl = i < a.nact ? P[i + 1] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            if (i < a.nact) P[i + 1] = run + incl;
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    __syncthreads();
    const int U = P[a.nact];
    const int G = (int)gridDim.x < U ? (int)gridDim.x : U;  // CTAs that get work
    const int cta = blockIdx.x;

    // segments that cannot take another row: report, write zeros
    for (int si = cta; si < a.nact; si += gridDim.x) {
        if (seg_rows[si] >= 0) continue;
        const int b = si / a.nl, seg = b * a.L + a.layer_begin + si % a.nl;
        if (tid == 0) raise_status(a.dev_status, b, PKV_DEV_CAPACITY);
        T *o = reinterpret_cast<T *>(a.out) + (size_t)seg * H * D;
        for (int e = tid; e < H * D; e += blockDim.x) o[e] = from_float<T>(0.f);
    }

    int u0 = 0, u1 = 0, si0 = 0;
    const int upc = G > 0 ? U / G : 0, rem = G > 0 ? U - upc * G : 0;
    // The merge kernel may be scheduled from here on; it still waits for this grid to finish.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (cta == 0) {
        // The plan, for the merge kernel: rows, first contributing CTA and number of contributing
        // CTAs of every active segment.  (That kernel must not rebuild it from len, which it bumps.)
        for (int i = tid; i < a.nact; i += blockDim.x) {
            const int rows = seg_rows[i];  // = the segment's length after this step
            int first = 0, cnt = 0;
            if (rows >= 0) {
                first = unit_owner(P[i], upc, rem);
                cnt = unit_owner(P[i + 1] - 1, upc, rem) - first + 1;
            }
            reinterpret_cast<int4 *>(a.plan)[i] = make_int4(rows, first, cnt, seg_dst[i]);
        }
    }
    if (cta < G) {
        u0 = first_unit(cta, upc, rem);
        u1 = first_unit(cta + 1, upc, rem);
        int lo = 0, hi = a.nact;  // last segment whose first unit is <= u0
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (P[mid] <= u0) lo = mid; else hi = mid;
        }
        si0 = lo;
    }

    if (warp == NW) {
        // ---- producer: the only thread that reads global memory while the stream runs --------
        if (lane == 0 && u0 < u1) {
            Ring r{0, a.nstages, 0u};
            int qi = 0;
            uint32_t qph = 0;
            int si = si0, issued = 0;
            bool dead = false, piece_start = true;
            int n = 0, r0 = 0, seg = 0, newrow = 0;
            int64_t off = 0;
            for (int u = u0; u < u1 && !dead; ++u) {
                if (u >= P[si + 1]) {
                    do ++si; while (u >= P[si + 1]);
                    piece_start = true;
                }
                if (piece_start) {
                    piece_start = false;
                    seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
                    n = seg_rows[si];
                    newrow = seg_dst[si] & 0x3fffffff;
                    off = seg_off[si];
                    r0 = (u - P[si]) * UR;
                    wait_phase(qempty + qi, qph ^ 1u, dead, &s_abort);
                    if (dead) break;
                    mbar_expect_tx(qfull + qi, rb);
                    bulk_load(qbuf + (size_t)qi * rb, reinterpret_cast<const unsigned char *>(a.q) + (size_t)seg * rb,
                              rb, qfull + qi);
                    qi ^= 1;
                    if (qi == 0) qph ^= 1u;
                }
                const int cnt = min(UR, n - r0);          // rows of this unit
                const int nd = newrow - r0;               // the new row's place in it, if 0 <= nd < cnt
                const bool has_new = nd >= 0 && nd < cnt;
                const int before = has_new ? nd : cnt;    // cached rows in front of it
                const int after = has_new ? cnt - nd - 1 : 0;  // and behind it (only when a slot is reused)
                const uint32_t bytes = (uint32_t)cnt * rb;
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {
                    wait_phase(empty + r.slot, r.phase ^ 1u, dead, &s_abort);
                    if (dead) break;
                    unsigned char *dst = ring + (size_t)r.slot * slot_bytes;
                    mbar_expect_tx(full + r.slot, bytes);
                    const unsigned char *cache = reinterpret_cast<const unsigned char *>(kv ? a.cv : a.ck);
                    if (before > 0)
                        bulk_load(dst, cache + (size_t)(off + r0) * rb, (uint32_t)before * rb, full + r.slot);
                    if (has_new)
                        bulk_load(dst + (size_t)nd * rb,
                                  reinterpret_cast<const unsigned char *>(kv ? a.v_new : a.k_new) + (size_t)seg * rb, rb,
                                  full + r.slot);
                    if (after > 0)
                        bulk_load(dst + (size_t)(nd + 1) * rb, cache + (size_t)(off + r0 + nd + 1) * rb,
                                  (uint32_t)after * rb, full + r.slot);
                    r.advance();
                    ++issued;
                }
                r0 += UR;
            }
            if (dead) {
                // let copies already issued land before the CTA can exit (bounded)
                for (int i = 0; i < a.nstages && i < issued; ++i) mbar_wait(full + i, 0u);
            }
        }
    } else if (u0 < u1) {
        // ---- consumers --------------------------------------------------------------------
        const int g = lane / LPR, c = lane % LPR;
        const int h0 = warp * HPW;  // H is a multiple of HPW (checked by the launcher)
        const uint32_t lane_off = (uint32_t)h0 * D * sizeof(T) + c * 16;
        // Four heads per warp in a block of more than 12 warps (96 registers per thread): q stays in its
        // shared-memory buffer for the piece and a head's slice is re-read for every unit, which keeps
        // that variant free of spills.  With fewer warps there is room for q in registers.
        constexpr bool kQSmem = HPW >= 4 && MAXT > 384;
        float qf[kQSmem ? 1 : HPW][kQSmem ? 1 : EPL], acc[HPW][EPL], m[HPW], l[HPW];
        const unsigned char *q_held = nullptr;
        int q_held_idx = 0;
        float q_scale = 0.f;
        Ring r{0, a.nstages, 0u};
        int qi = 0;
        uint32_t qph = 0;
        int si = si0;
        bool dead = false, piece_start = true;
        int n = 0, r0 = 0, seg = 0, seg_last_u = 0, newrow = 0;
        int64_t off = 0;
        size_t seg_vec = 0;
        for (int u = u0; u < u1; ++u) {
            if (u > seg_last_u && !piece_start) {
                piece_start = true;
            }
            if (piece_start) {
                piece_start = false;
                while (u >= P[si + 1]) ++si;
                seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
                n = seg_rows[si];
                newrow = seg_dst[si] & 0x3fffffff;
                off = seg_off[si];
                r0 = (u - P[si]) * UR;
                seg_last_u = P[si + 1] - 1;
                seg_vec = (size_t)seg * H * D;
                const float sc = a.layer_scale[a.layer_begin + si % a.nl] * kLog2eD;
                wait_phase(qfull + qi, qph, dead, &s_abort);
                const unsigned char *qb = qbuf + (size_t)qi * rb;
#pragma unroll
                for (int hh = 0; hh < HPW; ++hh) {
                    m[hh] = -INFINITY;
                    l[hh] = 0.f;
                    const int h = h0 + hh;
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        float x[VE];
                        Vec<T>::unpack(*reinterpret_cast<const uint4 *>(qb + (size_t)h * D * sizeof(T) + (v * LPR + c) * 16), x);
#pragma unroll
                        for (int i = 0; i < VE; ++i) {
                            if constexpr (!kQSmem) qf[hh][v * VE + i] = x[i] * sc;
                            acc[hh][v * VE + i] = 0.f;
                        }
                    }
                }
                if constexpr (kQSmem) {
                    q_held = qb + (size_t)h0 * D * sizeof(T) + c * 16;
                    q_held_idx = qi;
                    q_scale = sc;
                } else {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(qempty + qi);
                }
                qi ^= 1;
                if (qi == 0) qph ^= 1u;
            }
            const int cnt = min(UR, n - r0);      // rows of this unit, the new row included
            const int new_idx = newrow - r0;      // the new row's index in the unit when 0 <= new_idx < cnt
            const bool has_new = new_idx >= 0 && new_idx < cnt;
            const bool seg_end = u == seg_last_u;
            float s[HPW][RPG];
            const bool whole = cnt == UR;  // every row of the unit is valid (uniform over the CTA)

            // ---- K item: logits ---------------------------------------------------------------
            {
                wait_phase(full + r.slot, r.phase, dead, &s_abort);
                const unsigned char *kb = ring + (uint32_t)r.slot * slot_bytes;
                const unsigned char *kl = kb + (uint32_t)g * rb + lane_off;
                if constexpr (kQSmem) {
#pragma unroll
                    for (int hh = 0; hh < HPW; ++hh) {
                        float qv[EPL];  // this head's slice of the scaled query
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            float x[VE];
                            Vec<T>::unpack(*reinterpret_cast<const uint4 *>(q_held + hh * (int)(D * sizeof(T)) + v * LPR * 16), x);
#pragma unroll
                            for (int i = 0; i < VE; ++i) qv[v * VE + i] = x[i] * q_scale;
                        }
#pragma unroll
                        for (int j = 0; j < RPG; ++j) {
                            float d0 = 0.f, d1 = 0.f;
                            if (whole || g + j * GPW < cnt) {
                                const unsigned char *row = kl + (uint32_t)(j * GPW) * rb + hh * (int)(D * sizeof(T));
#pragma unroll
                                for (int v = 0; v < NV; ++v) {
                                    float x[VE];
                                    Vec<T>::unpack(*reinterpret_cast<const uint4 *>(row + v * LPR * 16), x);
#pragma unroll
                                    for (int i = 0; i < VE; i += 2) {
                                        d0 = fmaf(qv[v * VE + i], x[i], d0);
                                        d1 = fmaf(qv[v * VE + i + 1], x[i + 1], d1);
                                    }
                                }
                            }
                            s[hh][j] = d0 + d1;
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < RPG; ++j) {
#pragma unroll
                        for (int hh = 0; hh < HPW; ++hh) {
                            float d0 = 0.f, d1 = 0.f;
                            if (whole || g + j * GPW < cnt) {
                                const unsigned char *row = kl + (uint32_t)(j * GPW) * rb + hh * (int)(D * sizeof(T));
#pragma unroll
                                for (int v = 0; v < NV; ++v) {
                                    float x[VE];
                                    Vec<T>::unpack(*reinterpret_cast<const uint4 *>(row + v * LPR * 16), x);
#pragma unroll
                                    for (int i = 0; i < VE; i += 2) {
                                        d0 = fmaf(qf[hh][v * VE + i], x[i], d0);
                                        d1 = fmaf(qf[hh][v * VE + i + 1], x[i + 1], d1);
                                    }
                                }
                            }
                            s[hh][j] = d0 + d1;
                        }
                    }
                }
#pragma unroll
                for (int o = LPR / 2; o > 0; o >>= 1)
#pragma unroll
                    for (int j = 0; j < RPG; ++j)
#pragma unroll
                        for (int hh = 0; hh < HPW; ++hh) s[hh][j] += __shfl_xor_sync(0xffffffffu, s[hh][j], o);
                if (has_new) {  // this warp's heads of the new K row go to their cache row
                    const unsigned char *src = kb + (uint32_t)new_idx * rb + (uint32_t)h0 * D * sizeof(T);
                    unsigned char *dst = reinterpret_cast<unsigned char *>(a.ck) + (size_t)(off + newrow) * rb +
                                         (size_t)h0 * D * sizeof(T);
                    for (int x = lane; x < HPW * (int)(D * sizeof(T) / 16); x += 32)
                        *reinterpret_cast<uint4 *>(dst + x * 16) = *reinterpret_cast<const uint4 *>(src + x * 16);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty + r.slot);
                r.advance();
            }
            // ---- V item: softmax update (one rescale per unit) and accumulation -------------------
            {
#pragma unroll
                for (int hh = 0; hh < HPW; ++hh) {
                    float mx = m[hh];
#pragma unroll
                    for (int j = 0; j < RPG; ++j) {
                        if (!(whole || g + j * GPW < cnt)) s[hh][j] = -INFINITY;
                        mx = fmaxf(mx, s[hh][j]);
                    }
                    // mx stays -inf only for a group that has seen no row yet; keep its state at zero
                    const float corr = mx == -INFINITY ? 1.f : exp2f(m[hh] - mx);
                    m[hh] = mx;
                    float lsum = l[hh] * corr;
#pragma unroll
                    for (int j = 0; j < RPG; ++j) {
                        s[hh][j] = mx == -INFINITY ? 0.f : exp2f(s[hh][j] - mx);
                        lsum += s[hh][j];
                    }
                    l[hh] = lsum;
#pragma unroll
                    for (int i = 0; i < EPL; ++i) acc[hh][i] *= corr;
                }
                wait_phase(full + r.slot, r.phase, dead, &s_abort);
                const unsigned char *vb = ring + (uint32_t)r.slot * slot_bytes;
                const unsigned char *vl = vb + (uint32_t)g * rb + lane_off;
#pragma unroll
                for (int j = 0; j < RPG; ++j) {
#pragma unroll
                    for (int hh = 0; hh < HPW; ++hh) {
                        if (whole || g + j * GPW < cnt) {
                            const float pj = s[hh][j];
                            const unsigned char *row = vl + (uint32_t)(j * GPW) * rb + hh * (int)(D * sizeof(T));
#pragma unroll
                            for (int v = 0; v < NV; ++v) {
                                float x[VE];
                                Vec<T>::unpack(*reinterpret_cast<const uint4 *>(row + v * LPR * 16), x);
#pragma unroll
                                for (int i = 0; i < VE; ++i)
                                    acc[hh][v * VE + i] = fmaf(pj, x[i], acc[hh][v * VE + i]);
                            }
                        }
                    }
                }
                if (has_new) {
                    const unsigned char *src = vb + (uint32_t)new_idx * rb + (uint32_t)h0 * D * sizeof(T);
                    unsigned char *dst = reinterpret_cast<unsigned char *>(a.cv) + (size_t)(off + newrow) * rb +
                                         (size_t)h0 * D * sizeof(T);
                    for (int x = lane; x < HPW * (int)(D * sizeof(T) / 16); x += 32)
                        *reinterpret_cast<uint4 *>(dst + x * 16) = *reinterpret_cast<const uint4 *>(src + x * 16);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty + r.slot);
                r.advance();
            }
            r0 += UR;

            if (seg_end || u == u1 - 1) {
                // ---- close this CTA's piece of the segment ---------------------------------------
                if constexpr (kQSmem) {  // q was read in place until here
                    __syncwarp();
                    if (lane == 0) mbar_arrive(qempty + q_held_idx);
                }
                const int c_first = unit_owner(P[si], upc, rem), c_last = unit_owner(P[si + 1] - 1, upc, rem);
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
                piece_start = true;
            }
        }

        if (dead && lane == 0) raise_status(a.dev_status, 0, PKV_DEV_TIMEOUT);
    }

}

template <typename T, int E> struct Pack;
template <> struct Pack<float, 4> {
    __device__ static void store(float *dst, const float *x) { *reinterpret_cast<float4 *>(dst) = make_float4(x[0], x[1], x[2], x[3]); }
};
template <> struct Pack<float, 2> {
    __device__ static void store(float *dst, const float *x) { *reinterpret_cast<float2 *>(dst) = make_float2(x[0], x[1]); }
};
template <> struct Pack<__nv_bfloat16, 4> {
    __device__ static void store(__nv_bfloat16 *dst, const float *x)
    {
        __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]), b = __floats2bfloat162_rn(x[2], x[3]);
        *reinterpret_cast<uint2 *>(dst) =
            make_uint2(*reinterpret_cast<uint32_t *>(&a), *reinterpret_cast<uint32_t *>(&b));
    }
};
template <> struct Pack<__nv_bfloat16, 2> {
    __device__ static void store(__nv_bfloat16 *dst, const float *x)
    {
        *reinterpret_cast<__nv_bfloat162 *>(dst) = __floats2bfloat162_rn(x[0], x[1]);
    }
};
template <int E> struct LoadF;
template <> struct LoadF<4> {
    __device__ static void ld(const float *p, float *x)
    {
        const float4 v = __ldcg(reinterpret_cast<const float4 *>(p));
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
};
template <> struct LoadF<2> {
    __device__ static void ld(const float *p, float *x)
    {
        const float2 v = __ldcg(reinterpret_cast<const float2 *>(p));
        x[0] = v.x; x[1] = v.y;
    }
};

// Merge kernel, launched as a programmatic dependent of the stream kernel, whose CTA 0 leaves
// it one record per active segment (length after the step, first contributing CTA, number of
// contributors, row written).  Every block copies the records to shared memory and lists the
// segments that were split over several CTAs; its warps then take (split segment, group of HG
// heads) items in a grid-stride loop and combine the partials -- lane x holds elements
// [x * D / 32, (x + 1) * D / 32) of a head, and HG heads x KB contributors are in flight before
// any is used.  One thread per segment writes the new length.  Nothing here reads len: blocks of
// one grid start at different times.
constexpr int kFinishWarps = 16;
template <typename T, int D, int HG>
__global__ void __launch_bounds__(kFinishWarps * 32) decode_finish_kernel(const DecodeArgs a)
{
    constexpr int kSlotStride = D + 4, EPM = D / 32, KB = 8 / HG;
    __shared__ int4 rec[kMaxActive];
    __shared__ short split_seg[kMaxActive];
    __shared__ int nsplit;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // e.g. the next decode step
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the stream kernel's writes are visible
    for (int i = tid; i < a.nact; i += blockDim.x) rec[i] = reinterpret_cast<const int4 *>(a.plan)[i];
    __syncthreads();
    if (warp == 0) {  // the split segments, in order
        int n = 0;
        for (int base = 0; base < a.nact; base += 32) {
            const int i = base + lane;
            const bool is_split = i < a.nact && rec[i].x >= 0 && rec[i].z > 1;
            const unsigned m = __ballot_sync(0xffffffffu, is_split);
            if (is_split) split_seg[n + __popc(m & ((1u << lane) - 1))] = (short)i;
            n += __popc(m);
        }
        if (lane == 0) nsplit = n;
    }
    __syncthreads();

    for (int si = blockIdx.x * blockDim.x + tid; si < a.nact; si += gridDim.x * blockDim.x) {
        const int4 r = rec[si];
        if (r.x < 0) continue;  // could not take a row: reported and zero-filled by the stream kernel
        const int seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
        a.len[seg] = r.x;
        const int d = a.k_new ? a.evict_distance : 0;
        if (d > 0) {  // only this thread touches the segment's token count and slot ring
            const int g = a.gen[seg];
            int32_t *ring = a.slot_ring + (size_t)seg * (d + 1);
            if (r.w >> 30) ring[(g - d) % (d + 1)] = -1;  // the token d steps back gave up its slot
            ring[g % (d + 1)] = r.w & 0x3fffffff;
            a.gen[seg] = g + 1;
        }
    }

    const int groups = a.H / HG;
    const size_t cstride = (size_t)a.H * kSlotStride;
    for (int item = blockIdx.x * kFinishWarps + warp; item < nsplit * groups; item += gridDim.x * kFinishWarps) {
        const int sp = item / groups, h0 = (item - sp * groups) * HG;
        const int si = split_seg[sp];
        const int4 r = rec[si];
        const int c_first = r.y, ncontrib = r.z;
        const int seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
        const float *base = a.scratch + ((size_t)(c_first + si) * a.H + h0) * kSlotStride;
        float M[HG], z[HG], o[HG][EPM];
#pragma unroll
        for (int hh = 0; hh < HG; ++hh) {
            M[hh] = -INFINITY;
            z[hh] = 0.f;
#pragma unroll
            for (int i = 0; i < EPM; ++i) o[hh][i] = 0.f;
        }
#pragma unroll 1
        for (int k0 = 0; k0 < ncontrib; k0 += KB) {
            float2 ml[HG][KB];
            float x[HG][KB][EPM];
#pragma unroll
            for (int kk = 0; kk < KB; ++kk) {
                const float *sl = base + (size_t)min(k0 + kk, ncontrib - 1) * cstride;
#pragma unroll
                for (int hh = 0; hh < HG; ++hh) {
                    ml[hh][kk] = *reinterpret_cast<const float2 *>(sl + hh * kSlotStride + D);
                    LoadF<EPM>::ld(sl + hh * kSlotStride + lane * EPM, x[hh][kk]);
                }
            }
#pragma unroll
            for (int hh = 0; hh < HG; ++hh) {
                float mb = M[hh];
#pragma unroll
                for (int kk = 0; kk < KB; ++kk)
                    if (k0 + kk < ncontrib) mb = fmaxf(mb, ml[hh][kk].x);
                const float corr = M[hh] == -INFINITY ? 0.f : exp2f(M[hh] - mb);
                z[hh] *= corr;
#pragma unroll
                for (int i = 0; i < EPM; ++i) o[hh][i] *= corr;
                M[hh] = mb;
#pragma unroll
                for (int kk = 0; kk < KB; ++kk) {
                    if (k0 + kk < ncontrib) {
                        const float ww = exp2f(ml[hh][kk].x - mb);
                        z[hh] = fmaf(ww, ml[hh][kk].y, z[hh]);
#pragma unroll
                        for (int i = 0; i < EPM; ++i) o[hh][i] = fmaf(ww, x[hh][kk][i], o[hh][i]);
                    }
                }
            }
        }
#pragma unroll
        for (int hh = 0; hh < HG; ++hh) {
            const float inv = 1.f / z[hh];
#pragma unroll
            for (int i = 0; i < EPM; ++i) o[hh][i] *= inv;
            Pack<T, EPM>::store(reinterpret_cast<T *>(a.out) + ((size_t)seg * a.H + h0 + hh) * D + lane * EPM, o[hh]);
        }
    }
}

// Merge kernel for few segments: one warp per (active segment, head), no shared memory, no block
// barrier.  The segment's record is read twice: before griddepcontrol.wait (the stream kernel wrote
// it in its first microsecond, so this early copy is almost always the final one), so that the
// loads of the partials can go out the moment the wait returns, and again after it, in flight
// together with those loads.  The early copy's result is kept only if the two copies agree;
// otherwise the merge is redone from the second.  The early copy is never trusted for addresses
// beyond the slots that exist, nor for what is written to len.
template <typename T, int D>
__global__ void __launch_bounds__(kFinishWarps * 32) decode_finish_small_kernel(const DecodeArgs a, int nslots)
{
    constexpr int kSlotStride = D + 4, EPM = D / 32, KB = 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int item = blockIdx.x * kFinishWarps + warp;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // e.g. the next decode step
    if (item >= a.nact * a.H) return;
    const int si = item / a.H, h = item - si * a.H;
    const int4 *recp = reinterpret_cast<const int4 *>(a.plan) + si;
    const int4 early = __ldcg(recp);
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the stream kernel's writes are visible
    const int4 late = __ldcg(recp);
    const int seg = (si / a.nl) * a.L + a.layer_begin + si % a.nl;
    const size_t cstride = (size_t)a.H * kSlotStride;

    int4 r = early;
    float M = -INFINITY, z = 0.f, o[EPM];
    for (int attempt = 0; attempt < 2; ++attempt) {
        M = -INFINITY;
        z = 0.f;
#pragma unroll
        for (int i = 0; i < EPM; ++i) o[i] = 0.f;
        // (the early copy may be anything, e.g. what another shape's call left in the workspace:
        // bound each field before adding them, so that the sum cannot wrap)
        const bool usable = r.x >= 0 && r.y >= 0 && r.y < nslots && r.z > 1 && r.z <= nslots &&
                            r.y + si + r.z <= nslots;
        if (usable) {
            const int c_first = r.y, ncontrib = r.z;
            const float *base = a.scratch + ((size_t)(c_first + si) * a.H + h) * kSlotStride;
#pragma unroll 1
            for (int k0 = 0; k0 < ncontrib; k0 += KB) {
                float2 ml[KB];
                float x[KB][EPM];
#pragma unroll
                for (int kk = 0; kk < KB; ++kk) {
                    const float *sl = base + (size_t)min(k0 + kk, ncontrib - 1) * cstride;
                    ml[kk] = __ldcg(reinterpret_cast<const float2 *>(sl + D));
                    LoadF<EPM>::ld(sl + lane * EPM, x[kk]);
                }
                float mb = M;
#pragma unroll
                for (int kk = 0; kk < KB; ++kk)
                    if (k0 + kk < ncontrib) mb = fmaxf(mb, ml[kk].x);
                const float corr = M == -INFINITY ? 0.f : exp2f(M - mb);
                z *= corr;
#pragma unroll
                for (int i = 0; i < EPM; ++i) o[i] *= corr;
                M = mb;
#pragma unroll
                for (int kk = 0; kk < KB; ++kk) {
                    if (k0 + kk < ncontrib) {
                        const float ww = exp2f(ml[kk].x - mb);
                        z = fmaf(ww, ml[kk].y, z);
#pragma unroll
                        for (int i = 0; i < EPM; ++i) o[i] = fmaf(ww, x[kk][i], o[i]);
                    }
                }
            }
        }
        if (attempt == 1 || (late.x == r.x && late.y == r.y && late.z == r.z && late.w == r.w)) break;
        r = late;
    }
    // from here on r is the record as the finished stream kernel left it
    if (r.x < 0) return;  // could not take a row: reported and zero-filled by the stream kernel
    if (h == 0 && lane == 0) {
        a.len[seg] = r.x;
        const int d = a.k_new ? a.evict_distance : 0;
        if (d > 0) {  // only this thread touches the segment's token count and slot ring
            const int g = a.gen[seg];
            int32_t *ring = a.slot_ring + (size_t)seg * (d + 1);
            if (r.w >> 30) ring[(g - d) % (d + 1)] = -1;  // the token d steps back gave up its slot
            ring[g % (d + 1)] = r.w & 0x3fffffff;
            a.gen[seg] = g + 1;
        }
    }
    if (r.z <= 1) return;  // one CTA covered the segment and wrote its output
    const float inv = 1.f / z;
#pragma unroll
    for (int i = 0; i < EPM; ++i) o[i] *= inv;
    Pack<T, EPM>::store(reinterpret_cast<T *>(a.out) + ((size_t)seg * a.H + h) * D + lane * EPM, o);
}

static size_t plan_bytes(int nact) { return round_up((size_t)nact * sizeof(int4), kWsAlign); }

size_t decode_stream_ws_bytes(const pkv_shape *s)
{
    size_t nseg = (size_t)s->batch * s->layers;
    size_t slots = 256 + nseg;
    return plan_bytes((int)(nseg < (size_t)kMaxActive ? nseg : kMaxActive)) +
           round_up(slots * s->heads * (s->head_dim + 4) * sizeof(float), kWsAlign);
}

static size_t stream_smem_bytes(int nstages, int ur, uint32_t rb, int nact)
{
    return (size_t)nstages * ur * rb + 2 * (size_t)rb + (2 * kMaxStages + 4) * sizeof(uint64_t) +
           (size_t)nact * sizeof(int64_t) + (size_t)(3 * nact + 1) * sizeof(int) + 32;
}

template <typename T, int D, int LPR, int HPW, int UR, int MAXT>
static int launch_variant(const DecodeArgs &a, int sms, cudaStream_t st)
{
    static bool done[64] = {};
    if ((a.nwarps + 1) * 32 > MAXT) return -1;
    int rc = ensure_dynamic_smem((const void *)decode_stream_kernel<T, D, LPR, HPW, UR, MAXT>, kDynSmemMax, done);
    if (rc != PKV_OK) return rc;
    // Both kernels are programmatic dependents of their predecessor in the stream: they may be
    // set up while it still runs and go past their griddepcontrol.wait once it has completed.
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms);
    cfg.blockDim = dim3((a.nwarps + 1) * 32);
    cfg.dynamicSmemBytes = stream_smem_bytes(a.nstages, UR, a.row_bytes, a.nact);
    cfg.stream = st;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_stream_kernel<T, D, LPR, HPW, UR, MAXT>, a);
    if (e != cudaSuccess) {
        set_cuda_error(e, "decode_stream_kernel");
        return PKV_ERR_CUDA;
    }
    // One head per warp item while that still fills the GPU once (every partial of a segment is
    // then in flight at the same time); two heads per item beyond that.
    const int hg = (a.H % 2 == 0 && a.nact * a.H > sms * kFinishWarps) ? 2 : 1;
    const int items = a.nact * (a.H / hg);
    const int blocks = (items + kFinishWarps - 1) / kFinishWarps;
    cfg.gridDim = dim3(blocks < sms ? blocks : sms);
    cfg.blockDim = dim3(kFinishWarps * 32);
    cfg.dynamicSmemBytes = 0;
    if (hg == 2) {
        e = cudaLaunchKernelEx(&cfg, decode_finish_kernel<T, D, 2>, a);
    } else if (items <= sms * kFinishWarps) {  // a warp for every (segment, head): the barrier-free kernel
        cfg.gridDim = dim3(blocks);
        const int nslots = 256 + a.nseg_total;  // partial slots the workspace holds
        e = cudaLaunchKernelEx(&cfg, decode_finish_small_kernel<T, D>, a, nslots);
    } else {
        e = cudaLaunchKernelEx(&cfg, decode_finish_kernel<T, D, 1>, a);
    }
    if (e != cudaSuccess) {
        set_cuda_error(e, "decode_finish_kernel");
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

// Returns PKV_OK, an error, or -1 when this shape is outside what the streaming kernel covers.
int launch_decode_stream(const pkv_shape *s, pkv_cache *c, const void *q, const void *kn,
                         const void *vn, const float *scale, int lb, int le, void *out,
                         int32_t *dev_status, void *ws, cudaStream_t st)
{
    const int H = s->heads, D = s->head_dim, nl = le - lb, nact = s->batch * nl;
    if (nact > kMaxActive || H > 64) return -1;
    const size_t es = esize(s);
    const uint32_t row_bytes = (uint32_t)((size_t)H * D * es);
    int ur = 0, nstages = 0;
    for (int cand = 8; cand >= 2 && !ur; cand >>= 1) {  // rows per unit: as many as leave three ring stages
        int ns = kMaxStages;
        while (ns >= 3 && stream_smem_bytes(ns, cand, row_bytes, nact) > (size_t)kDynSmemMax) --ns;
        if (ns >= 3) {
            ur = cand;
            nstages = ns;
        }
    }
    if (!ur) return -1;

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
    a.row_offset = c->row_offset; a.len = c->len; a.cap = c->cap;
    a.layer_scale = scale; a.dev_status = dev_status;
    a.plan = (int *)ws;
    a.scratch = (float *)((unsigned char *)ws + plan_bytes(nact));
    a.L = s->layers; a.H = H; a.layer_begin = lb; a.nl = nl; a.nact = nact;
    a.nseg_total = s->batch * s->layers; a.nstages = nstages; a.row_bytes = row_bytes;
    a.total_cap_rows = c->total_cap_rows;
    a.evict_distance = c->evict_distance;
    a.len0 = c->len0; a.gen = c->gen; a.slot_ring = c->slot_ring;
    a.N = s->prompt_len;

    const bool bf = s->dtype == PKV_BF16;
    const int vec_per_head = D / (int)(16 / es);
    // (lanes per row, heads per warp): at most 17 warps, and few enough registers of per-head
    // state that each SM sub-partition's register file holds its warps.  (The last template
    // argument is the block-size bound a variant is compiled for: 9, 12 or 17 warps, the smaller
    // ones with room for more registers per thread.)
    int lpr = 8, hpw = H <= 16 ? 1 : (H <= 32 ? 2 : 4);
    if (H > 16 && vec_per_head >= 16) lpr = 16;
    if (vec_per_head < lpr || H % hpw != 0) return -1;
    a.nwarps = H / hpw;
#define PKV_V(T, DD, LPR, HPW, UR, MAXT)                                       \
    if (lpr == LPR && hpw == HPW && ur == UR && (a.nwarps + 1) * 32 <= MAXT) \
        return launch_variant<T, DD, LPR, HPW, UR, MAXT>(a, sms, st)
    // Only what the choice above can ask for is instantiated: eight lanes per row with one head per
    // warp (at most 16 heads) for every type; with more heads per warp only where a head row has
    // fewer than sixteen 16-byte vectors (bf16, D = 64); sixteen lanes per row otherwise.  Four
    // heads per warp means more than 32 heads, i.e. at least ten warps.
#define PKV_NARROW1(T, DD)      \
    PKV_V(T, DD, 8, 1, 8, 544); \
    PKV_V(T, DD, 8, 1, 4, 544)
#define PKV_NARROW(T, DD)       \
    PKV_V(T, DD, 8, 2, 8, 544); \
    PKV_V(T, DD, 8, 4, 8, 384); \
    PKV_V(T, DD, 8, 4, 8, 544); \
    PKV_V(T, DD, 8, 2, 4, 544); \
    PKV_V(T, DD, 8, 4, 4, 384); \
    PKV_V(T, DD, 8, 4, 4, 544)
#define PKV_WIDE(T, DD)          \
    PKV_V(T, DD, 16, 2, 8, 544); \
    PKV_V(T, DD, 16, 4, 8, 384); \
    PKV_V(T, DD, 16, 4, 8, 544); \
    PKV_V(T, DD, 16, 2, 4, 544); \
    PKV_V(T, DD, 16, 4, 4, 384); \
    PKV_V(T, DD, 16, 4, 4, 544); \
    PKV_V(T, DD, 16, 2, 2, 544); \
    PKV_V(T, DD, 16, 4, 2, 384); \
    PKV_V(T, DD, 16, 4, 2, 544)
    if (bf && D == 128) {
        PKV_NARROW1(__nv_bfloat16, 128);
        PKV_WIDE(__nv_bfloat16, 128);
    } else if (bf && D == 64) {
        PKV_NARROW1(__nv_bfloat16, 64);
        PKV_NARROW(__nv_bfloat16, 64);
    } else if (!bf && D == 128) {
        PKV_NARROW1(float, 128);
        PKV_WIDE(float, 128);
    } else if (!bf && D == 64) {
        PKV_NARROW1(float, 64);
        PKV_WIDE(float, 64);
    }
#undef PKV_NARROW1
#undef PKV_NARROW
#undef PKV_WIDE
#undef PKV_V
    return -1;
}

}  // namespace pkv

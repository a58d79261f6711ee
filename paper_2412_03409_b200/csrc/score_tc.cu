// Importance score (Sec. 3.2), tensor-core path for bf16 inputs.
//
//   pass 1: per query m, log2-sum-exp of the scaled causal logits over keys j <= m
//   pass 2: per key n, sum over queries m >= n of exp2(logit - lse[m])
//   then the mean over heads in index order (shared with the FP32 path)
//
// Both passes walk 128 x 128 logit tiles of one (sample, layer, head).  The tile is one
// tcgen05.mma chain (M = N = 128, K = 16 x D/16) whose operands TMA stages in shared memory
// with the 128-byte swizzle and whose fp32 accumulator lives in tensor memory.  The operand
// that stays for a whole work item supplies the accumulator's lanes: queries in pass 1, so a
// thread owns one query row and keeps its running max / sum in registers; keys in pass 2, so
// a thread owns one key and its column sum needs no cross-thread reduction or atomics.
//
// Roles per CTA (192 threads): warp 0 lane 0 issues TMA, warp 1 owns tensor memory and its
// lane 0 issues the MMAs, warps 2-5 read the accumulator (tcgen05.ld, one TMEM lane quarter
// per warp) and do the exponentials.  Two accumulators alternate so that the MMAs of tile
// j + 1 overlap the exponentials of tile j; two CTAs share an SM.  Work items (one stationary
// tile and the tiles streamed against it) come from a device counter: the TMA thread takes the
// next number and announces it to the other roles through a four-entry shared-memory queue,
// so CTAs that run faster do more.  Every mbarrier wait is bounded: when one runs out the CTA
// stops waiting, sets the call's abort word (the head mean then writes NaN for every score, which
// the selection stage reports as PKV_DEV_BAD_SCORE) and still releases its tensor memory.
#include <cuda.h>

#include "common.cuh"

namespace pkv {

namespace {

constexpr int TT = 128;            // tile side
constexpr int kStagesB = 2;        // streamed-operand stages
constexpr uint32_t kSpin = 1u << 20;       // tries per wait; each may sleep up to kSuspendNs
constexpr uint32_t kSuspendNs = 2000;      // suspend-time hint of one try: a waiting thread leaves the issue slots alone
constexpr float kLog2eT = 1.4426950408889634f;

struct ScoreArgs {
    const float *layer_scale;
    float *lse2;     // [B*L*H][Npad] log2-sum-exp of scaled logits, +inf beyond N
    float *partial;  // [B*L*H][N] per-head column sums
    int32_t *abort_word;  // device word set when a bounded wait runs out: the head mean then writes NaN scores
    int *next_item;       // [2] work counters, one per pass; zeroed, with the abort word, before the first pass
    int L, H, N, Npad, tiles, nseg;
};

__device__ __forceinline__ uint32_t saddr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(saddr(bar)), "r"(count));
}
__device__ __forceinline__ void bar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(saddr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(saddr(bar)) : "memory");
}
__device__ __forceinline__ bool bar_try(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(saddr(bar)), "r"(parity), "r"(kSuspendNs)
        : "memory");
    return ok != 0;
}
// Bounded wait.  `dead` latches for the calling thread once any wait in the CTA has run out.
__device__ __forceinline__ void bar_wait(uint64_t *bar, uint32_t parity, bool &dead, int *abort_flag,
                                         uint32_t limit = kSpin)
{
    if (dead) return;
    for (uint32_t i = 0; i < limit; ++i) {
        if (bar_try(bar, parity)) return;
        if ((i & 255u) == 255u && *(volatile int *)abort_flag) break;
    }
    dead = true;
    atomicExch(abort_flag, 1);
}

__device__ __forceinline__ void tma_load_5d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1,
                                            int c2, int c3, int c4)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(saddr(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(saddr(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}

// Shared-memory matrix descriptor, K-major operand with the 128-byte swizzle: rows of 128 bytes,
// eight-row groups 1024 bytes apart, tile base aligned to 1024 bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);  // start address, bits [0,14)
    d |= (uint64_t)1 << 16;                   // leading byte offset (not used by swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;         // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                   // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                   // layout type: 128-byte swizzle
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = N = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TT >> 3) << 17) |
                            ((uint32_t)(TT >> 4) << 24);

__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(saddr(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float (&v)[64])
{
    uint32_t r[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
// Both halves of a 128-column accumulator row: two loads in flight, one wait.
__device__ __forceinline__ void tmem_ld128(uint32_t taddr, float (&v)[128])
{
    uint32_t r[64], q[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr));
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : "=r"(q[0]), "=r"(q[1]), "=r"(q[2]), "=r"(q[3]), "=r"(q[4]), "=r"(q[5]), "=r"(q[6]), "=r"(q[7]), "=r"(q[8]), "=r"(q[9]), "=r"(q[10]), "=r"(q[11]), "=r"(q[12]), "=r"(q[13]), "=r"(q[14]), "=r"(q[15]), "=r"(q[16]), "=r"(q[17]), "=r"(q[18]), "=r"(q[19]), "=r"(q[20]), "=r"(q[21]), "=r"(q[22]), "=r"(q[23]), "=r"(q[24]), "=r"(q[25]), "=r"(q[26]), "=r"(q[27]), "=r"(q[28]), "=r"(q[29]), "=r"(q[30]), "=r"(q[31]), "=r"(q[32]), "=r"(q[33]), "=r"(q[34]), "=r"(q[35]), "=r"(q[36]), "=r"(q[37]), "=r"(q[38]), "=r"(q[39]), "=r"(q[40]), "=r"(q[41]), "=r"(q[42]), "=r"(q[43]), "=r"(q[44]), "=r"(q[45]), "=r"(q[46]), "=r"(q[47]), "=r"(q[48]), "=r"(q[49]), "=r"(q[50]), "=r"(q[51]), "=r"(q[52]), "=r"(q[53]), "=r"(q[54]), "=r"(q[55]), "=r"(q[56]), "=r"(q[57]), "=r"(q[58]), "=r"(q[59]), "=r"(q[60]), "=r"(q[61]), "=r"(q[62]), "=r"(q[63])
        : "r"(taddr + 64));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 64; ++i) {
        v[i] = __uint_as_float(r[i]);
        v[64 + i] = __uint_as_float(q[i]);
    }
}
// 2^x on the special-function unit, one instruction (inputs here are <= 0 or -inf; flushing
// denormal results to zero is harmless for sums of probabilities).
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }

struct Ring2 {
    int idx;
    uint32_t phase;
    __device__ __forceinline__ void next(int n)
    {
        if (++idx == n) {
            idx = 0;
            phase ^= 1u;
        }
    }
};

// Pass 1 on NC consecutive logits of one query row: running maximum and sum in the log2
// domain.  Four interleaved chains each for the maximum and the sum: with two reader warps per
// scheduler a long dependent chain would leave it idle.  `fast` (scale > 0, the usual case):
// the extreme of sc * x is sc * max x, so masked logits may stay -inf.
template <int NC>
__device__ __forceinline__ void lse_block(float (&v)[NC], float sc, bool fast, float &run_max, float &run_sum)
{
    if (!fast) {
#pragma unroll
        for (int i = 0; i < NC; ++i) v[i] = v[i] == -INFINITY ? -INFINITY : v[i] * sc;
    }
    // (three-input maximum: half the comparisons; the loop takes four values at a time, the last two come at the end)
    float c2[2] = {v[0], v[1]};
#pragma unroll
    for (int i = 2; i + 2 < NC; i += 4) {
        c2[0] = max3(c2[0], v[i], v[i + 1]);
        c2[1] = max3(c2[1], v[i + 2], v[i + 3]);
    }
    const float cmax = max3(c2[0], c2[1], fmaxf(v[NC - 2], v[NC - 1]));
    const float nm = fmaxf(run_max, fast ? cmax * sc : cmax);  // finite: column 0 is never masked
    float p4[4] = {0.f, 0.f, 0.f, 0.f};
    if (fast) {
#pragma unroll
        for (int i = 0; i < NC; ++i) p4[i & 3] += ex2(fmaf(v[i], sc, -nm));
    } else {
#pragma unroll
        for (int i = 0; i < NC; ++i) p4[i & 3] += ex2(v[i] - nm);
    }
    run_sum = fmaf(run_sum, ex2(run_max - nm), (p4[0] + p4[1]) + (p4[2] + p4[3]));
    run_max = nm;
}

// Pass 2 on the logits of NC consecutive queries against one key: sum of the probabilities,
// lse = the queries' normalisers (shared memory, log2 domain).  On the block the causal boundary
// crosses (`edge`) query i of the block counts only when i >= lane.
template <int NC>
__device__ __forceinline__ float colsum_block(const float (&v)[NC], const float *lse, float sc, bool edge, int lane)
{
    const float4 *lp = reinterpret_cast<const float4 *>(lse);
    float p4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i4 = 0; i4 < NC / 4; ++i4) {
        const float4 ls = lp[i4];
        const float lv[4] = {ls.x, ls.y, ls.z, ls.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i4 * 4 + u;
            const float p = ex2(fmaf(v[i], sc, -lv[u]));
            p4[u] += (!edge || i >= lane) ? p : 0.f;
        }
    }
    return (p4[0] + p4[1]) + (p4[2] + p4[3]);
}

// Work item w -> (segment-head sh, tile t).  CTAs take items in order from a counter.  The tiles
// of one head are consecutive items, so the CTAs running at any moment share a few dozen heads
// whose Q and K stay in L2 and every operand byte comes from HBM once per pass; within a head
// the longest item comes first (pass 1: the last query tile, pass 2: the first key tile), so
// that what is left for the end of the pass is short.  Pass 2 walks the heads backwards: it
// starts on what pass 1 touched last.
template <int PASS> __device__ __forceinline__ void decode_item(int w, int nsh, int tiles, int &sh, int &t)
{
    const int q = w / tiles, r = w - q * tiles;
    t = PASS == 1 ? tiles - 1 - r : r;
    sh = PASS == 1 ? q : nsh - 1 - q;
}

constexpr int kItemQ = 4;  // item numbers in flight between the loader and the other roles

// PASS 1: stationary = Q tile t, streamed = K tiles 0..t.  PASS 2: stationary = K tile t,
// streamed = Q tiles t..tiles-1.
template <int PASS, int D>
__global__ void __launch_bounds__(192, 2)
score_tile_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const ScoreArgs a)
{
    constexpr int KH = D / 64;                  // 128-byte swizzle atoms along the head dimension
    constexpr uint32_t HALF = TT * 128;         // bytes of one [128 rows x 64 elements] box
    constexpr uint32_t TILE = KH * HALF;        // bytes of one operand tile
    extern __shared__ unsigned char smem_raw[];
    unsigned char *base = reinterpret_cast<unsigned char *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *sA = base;
    unsigned char *sB = base + TILE;
    uint64_t *bars = reinterpret_cast<uint64_t *>(sB + kStagesB * TILE);
    uint64_t *a_full = bars, *a_empty = bars + 1, *b_full = bars + 2, *b_empty = b_full + kStagesB;
    uint64_t *s_full = b_empty + kStagesB, *s_empty = s_full + 2;
    uint64_t *q_full = s_empty + 2, *q_empty = q_full + kItemQ;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_empty + kItemQ);
    __shared__ int s_abort;
    __shared__ int q_item[kItemQ];  // the loader's announcements: an item number, or -1 for the end
    __shared__ __align__(16) float s_lse[2][4][TT];  // [accumulator][reader warp][query of the tile]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const CUtensorMap *map_stat = PASS == 1 ? &map_q : &map_k;
    const CUtensorMap *map_strm = PASS == 1 ? &map_k : &map_q;
    const int nsh = a.nseg * a.H;
    const int nitems = nsh * a.tiles;

    if (tid == 0) {
        s_abort = 0;
        bar_init(a_full, 1);
        bar_init(a_empty, 1);
        for (int i = 0; i < kStagesB; ++i) {
            bar_init(b_full + i, 1);
            bar_init(b_empty + i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            bar_init(s_full + i, 1);
            bar_init(s_empty + i, 4);
        }
        for (int i = 0; i < kItemQ; ++i) {
            bar_init(q_full + i, 1);
            bar_init(q_empty + i, 5);  // the MMA thread and the four reader warps
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // two 128-column fp32 accumulators
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(saddr(tmem_slot)),
                     "r"(256u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Launched as a programmatic dependent: everything above (barriers, tensor memory) was set up
    // while the kernel before it drained; its results (Q, K, the normalisers) are read from here on.
    dependent_entry();

    if (warp == 0) {
        // ---- TMA producer ---------------------------------------------------------------------
        if (lane == 0) {
            bool dead = false;
            uint32_t a_phase = 0;
            Ring2 rb{0, 0u}, rq{0, 0u};
            int *ctr = a.next_item + (PASS - 1);
            int next = atomicAdd(ctr, 1);  // asked for one item ahead: the answer takes a microsecond
            for (;;) {
                const int w = next < nitems ? next : -1;
                if (w >= 0) next = atomicAdd(ctr, 1);
                bar_wait(q_empty + rq.idx, rq.phase ^ 1u, dead, &s_abort);
                if (dead) break;
                q_item[rq.idx] = w;
                bar_arrive(q_full + rq.idx);
                rq.next(kItemQ);
                if (w < 0) break;
                int sh, t;
                decode_item<PASS>(w, nsh, a.tiles, sh, t);
                const int seg = sh / a.H, h = sh - seg * a.H, b = seg / a.L, l = seg - b * a.L;
                bar_wait(a_empty, a_phase ^ 1u, dead, &s_abort);
                if (dead) break;
                bar_expect_tx(a_full, TILE);
#pragma unroll
                for (int kh = 0; kh < KH; ++kh)
                    tma_load_5d(sA + kh * HALF, map_stat, a_full, kh * 64, t * TT, h, l, b);
                a_phase ^= 1u;
                const int j0 = PASS == 1 ? 0 : t, j1 = PASS == 1 ? t : a.tiles - 1;
                for (int j = j0; j <= j1; ++j) {
                    bar_wait(b_empty + rb.idx, rb.phase ^ 1u, dead, &s_abort);
                    if (dead) break;
                    bar_expect_tx(b_full + rb.idx, TILE);
#pragma unroll
                    for (int kh = 0; kh < KH; ++kh)
                        tma_load_5d(sB + rb.idx * TILE + kh * HALF, map_strm, b_full + rb.idx, kh * 64, j * TT, h, l, b);
                    rb.next(kStagesB);
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer -------------------------------------------------------------------------
        if (lane == 0) {
            bool dead = false;
            uint32_t a_phase = 0;
            Ring2 rb{0, 0u}, rs{0, 0u}, rq{0, 0u};
            for (;;) {
                bar_wait(q_full + rq.idx, rq.phase, dead, &s_abort);
                if (dead) break;
                const int w = q_item[rq.idx];
                bar_arrive(q_empty + rq.idx);
                rq.next(kItemQ);
                if (w < 0) break;
                int sh, t;
                decode_item<PASS>(w, nsh, a.tiles, sh, t);
                bar_wait(a_full, a_phase, dead, &s_abort);
                a_phase ^= 1u;
                const int count = PASS == 1 ? t + 1 : a.tiles - t;
                for (int jj = 0; jj < count && !dead; ++jj) {
                    bar_wait(b_full + rb.idx, rb.phase, dead, &s_abort);
                    bar_wait(s_empty + rs.idx, rs.phase ^ 1u, dead, &s_abort);
                    if (dead) break;
                    fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)rs.idx * TT;
                    const uint32_t a_addr = saddr(sA), b_addr = saddr(sB + rb.idx * TILE);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t off = (uint32_t)(k / 4) * HALF + (uint32_t)(k % 4) * 32;
                        mma_bf16(d_tmem, smem_desc(a_addr + off), smem_desc(b_addr + off), k > 0 ? 1u : 0u);
                    }
                    mma_commit(b_empty + rb.idx);  // the streamed stage is free once these MMAs retire
                    mma_commit(s_full + rs.idx);   // and the accumulator is ready to be read
                    rb.next(kStagesB);
                    rs.next(2);
                }
                if (!dead) mma_commit(a_empty);     // the stationary tile may be replaced
            }
        }
    } else {
        // ---- accumulator readers: one TMEM lane (tile row) per thread ----------------------------
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        bool dead = false;
        Ring2 rs{0, 0u}, rq{0, 0u};
        for (;;) {
            bar_wait(q_full + rq.idx, rq.phase, dead, &s_abort);
            if (dead) break;
            const int w = q_item[rq.idx];
            __syncwarp();
            if (lane == 0) bar_arrive(q_empty + rq.idx);
            rq.next(kItemQ);
            if (w < 0) break;
            int sh, t;
            decode_item<PASS>(w, nsh, a.tiles, sh, t);
            const int seg = sh / a.H, l = seg % a.L;
            const float sc = a.layer_scale[l] * kLog2eT;
            const bool fast = sc > 0.f;     // the usual case: the extreme of sc * x is sc * max x
            const int grow = t * TT + row;  // query (pass 1) or key (pass 2) index of this thread
            const float *lse_row = a.lse2 + (size_t)sh * a.Npad;
            float run_max = -INFINITY, run_sum = 0.f;  // pass 1
            float col_sum = 0.f;                       // pass 2
            const int j0 = PASS == 1 ? 0 : t, j1 = PASS == 1 ? t : a.tiles - 1;
            // pass 2: every thread needs the tile's 128 query normalisers.  Each warp keeps its own copy
            // in shared memory (four per lane, fetched a tile ahead so that the load's latency is not
            // in the way), so the reader warps never wait for one another.
            float4 lse_mine = make_float4(0.f, 0.f, 0.f, 0.f);
            if (PASS == 2) lse_mine = __ldg(reinterpret_cast<const float4 *>(lse_row + j0 * TT) + lane);
            for (int j = j0; j <= j1; ++j) {
                if (PASS == 2) {
                    __syncwarp();  // the warp is done with the copy this one replaces (two tiles back)
                    reinterpret_cast<float4 *>(s_lse[rs.idx][quarter])[lane] = lse_mine;
                    if (j < j1) lse_mine = __ldg(reinterpret_cast<const float4 *>(lse_row + (j + 1) * TT) + lane);
                    __syncwarp();
                }
                bar_wait(s_full + rs.idx, rs.phase, dead, &s_abort);
                fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)rs.idx * TT;
                const bool diag = j == t;
                // On the diagonal tile only the 32-column blocks that reach this warp's rows matter:
                // blocks 0..quarter in pass 1 (keys <= query), quarter..3 in pass 2 (queries >= key).
                const int c_lo = (PASS == 2 && diag) ? quarter : 0;
                const int c_hi = (PASS == 1 && diag) ? quarter : TT / 32 - 1;
                bool released = false;
                if (!diag) {
                    // a full tile: the whole row comes into registers at once and the accumulator goes
                    // back to the MMA thread before the arithmetic starts
                    if (PASS == 1) {
                        float v[128];
                        tmem_ld128(taddr, v);
                        fence_before();
                        __syncwarp();
                        if (lane == 0) bar_arrive(s_empty + rs.idx);
                        released = true;
                        lse_block<128>(v, sc, fast, run_max, run_sum);
                    } else {  // (pass 2 keeps more state: half a row at a time fits its registers)
#pragma unroll 1
                        for (int half = 0; half < 2; ++half) {
                            float v[64];
                            tmem_ld64(taddr + half * 64, v);
                            if (half == 1) {
                                fence_before();
                                __syncwarp();
                                if (lane == 0) bar_arrive(s_empty + rs.idx);
                                released = true;
                            }
                            col_sum += colsum_block<64>(v, &s_lse[rs.idx][quarter][half * 64], sc, false, lane);
                        }
                    }
                } else {
#pragma unroll 1
                    for (int cblk = c_lo; cblk <= c_hi; ++cblk) {
                        float v[32];
                        tmem_ld32(taddr + cblk * 32, v);
                        const bool edge = cblk == quarter;  // the block the causal boundary crosses
                        if (PASS == 1) {
                            if (edge) {
#pragma unroll
                                for (int i = 0; i < 32; ++i) v[i] = i <= lane ? v[i] : -INFINITY;
                            }
                            lse_block<32>(v, sc, fast, run_max, run_sum);
                        } else {
                            col_sum += colsum_block<32>(v, &s_lse[rs.idx][quarter][cblk * 32], sc, edge, lane);
                        }
                    }
                }
                if (!released) {
                    fence_before();
                    __syncwarp();
                    if (lane == 0) bar_arrive(s_empty + rs.idx);
                }
                rs.next(2);
            }
            if (PASS == 1) {
                a.lse2[(size_t)sh * a.Npad + grow] = grow < a.N ? run_max + log2f(run_sum) : INFINITY;
            } else if (grow < a.N) {
                a.partial[(size_t)sh * a.N + grow] = col_sum;
            }
        }
    }
    // Any role whose wait ran out has set s_abort; one thread passes it on (after the barrier below).

    fence_before();
    __syncthreads();
    fence_after();
    if (tid == 0 && s_abort && a.abort_word) atomicExch(a.abort_word, (int)PKV_DEV_TIMEOUT);
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
    }
}

// One warp waits, with a short limit, on a barrier phase that nothing completes: the wait gives
// up, latches `dead`, and the status word reads PKV_DEV_TIMEOUT.  This is the whole give-up path
// of the kernel above in isolation (its roles then stop waiting, drain and release tensor memory).
__global__ void selftest_wait_kernel(int32_t *dev_status, uint32_t limit)
{
    __shared__ uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        bar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool dead = false;
    if (threadIdx.x == 0) bar_wait(&bar, 0u, dead, &s_abort, limit);
    __syncthreads();
    bar_wait(&bar, 0u, dead, &s_abort, limit);  // the other lanes see the flag and stop at once
    if (threadIdx.x == 0 && dead && s_abort) raise_status(dev_status, 0, PKV_DEV_TIMEOUT);
}

// Caller-supplied natural-log lse [B*L*H][N] -> padded log2 layout.
__global__ void convert_lse_kernel(const float *__restrict__ lse, int N, int Npad, size_t rows,
                                   float *__restrict__ lse2)
{
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows * Npad) return;
    size_t r = i / Npad;
    int n = (int)(i - r * Npad);
    lse2[i] = n < N ? lse[r * N + n] * kLog2eT : INFINITY;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// [B, L, H, N, D] bf16 with element strides -> rank-5 map, box = 64 elements x 128 rows.
bool make_map(CUtensorMap *map, const void *ptr, const pkv_shape *s, pkv_strides st)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[5] = {(cuuint64_t)s->head_dim, (cuuint64_t)s->prompt_len, (cuuint64_t)s->heads,
                          (cuuint64_t)s->layers, (cuuint64_t)s->batch};
    int64_t es[4] = {st.n, st.h, st.l, st.b};
    cuuint64_t strides[4];
    for (int i = 0; i < 4; ++i) {
        int64_t v = es[i];
        if (dims[i + 1] == 1 && v == 0) v = s->head_dim;  // a size-1 dimension's stride is never used
        strides[i] = (cuuint64_t)v * 2;
        if (strides[i] % 16 != 0 || strides[i] >= ((cuuint64_t)1 << 40) || strides[i] == 0) return false;
    }
    cuuint32_t box[5] = {64, TT, 1, 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int PASS, int D>
int launch_pass(const CUtensorMap &mq, const CUtensorMap &mk, const ScoreArgs &a, int sms, cudaStream_t st)
{
    static bool done[64] = {};
    const size_t smem = (size_t)(1 + kStagesB) * (D / 64) * TT * 128 + 1024 + 256;
    int rc = ensure_dynamic_smem((const void *)score_tile_kernel<PASS, D>, (int)smem, done);
    if (rc != PKV_OK) return rc;
    const int items = a.nseg * a.H * a.tiles;
    // CTAs take items from a counter as they finish (long and short items mix in any case; with a
    // fixed stride, 296 CTAs and 16 tiles per head left every CTA two tile indices only, and the
    // slowest did 12 tiles per item against a mean of 8.5).
    const int grid = items < 2 * sms ? items : 2 * sms;
    cudaError_t e = launch_dependent(score_tile_kernel<PASS, D>, dim3(grid), dim3(192), smem, st, mq, mk, a);
    if (e != cudaSuccess) {
        set_cuda_error(e, PASS == 1 ? "score_tile_kernel<1>" : "score_tile_kernel<2>");
        return PKV_ERR_CUDA;
    }
    return PKV_OK;
}

}  // namespace

int launch_head_mean(const float *partial, int H, int N, size_t total, float *scores, const int32_t *abort_word,
                     cudaStream_t st);

int selftest_wait_score(int32_t *dev_status, cudaStream_t st)
{
    selftest_wait_kernel<<<1, 32, 0, st>>>(dev_status, 2000u);  // each try may sleep up to kSuspendNs
    return check_launch("selftest_wait_kernel");
}

bool score_tc_usable(const pkv_shape *s, const void *, pkv_strides, const void *, pkv_strides)
{
    return s->dtype == PKV_BF16 && (s->head_dim == 64 || s->head_dim == 128) && encode_fn() != nullptr;
}

size_t score_tc_ws_bytes(const pkv_shape *s)
{
    const size_t rows = (size_t)s->batch * s->layers * s->heads;
    const size_t npad = ((size_t)s->prompt_len + TT - 1) / TT * TT;
    return round_up(rows * s->prompt_len * sizeof(float), kWsAlign) + round_up(rows * npad * sizeof(float), kWsAlign) +
           kWsAlign;  // the two work counters and the abort word
}

// Returns PKV_OK, an error, or -1 when the tensor maps cannot describe the caller's layout.
int launch_score_tc(const pkv_shape *s, const void *q, pkv_strides qs, const void *k, pkv_strides ks,
                    const float *scale, const float *lse, float *scores, void *ws, cudaStream_t st)
{
    CUtensorMap mq, mk;
    if (!make_map(&mq, q, s, qs) || !make_map(&mk, k, s, ks)) return -1;
    const int B = s->batch, L = s->layers, H = s->heads, N = s->prompt_len;
    const size_t rows = (size_t)B * L * H;
    ScoreArgs a;
    a.layer_scale = scale;
    a.partial = (float *)ws;
    a.lse2 = (float *)((unsigned char *)ws + round_up(rows * N * sizeof(float), kWsAlign));
    a.L = L; a.H = H; a.N = N;
    a.tiles = (N + TT - 1) / TT;
    a.Npad = a.tiles * TT;
    a.next_item = (int *)((unsigned char *)a.lse2 + round_up(rows * a.Npad * sizeof(float), kWsAlign));
    a.abort_word = a.next_item + 2;
    {
        cudaError_t e = cudaMemsetAsync(a.next_item, 0, 4 * sizeof(int), st);
        if (e != cudaSuccess) {
            set_cuda_error(e, "cudaMemsetAsync(score work counters)");
            return PKV_ERR_CUDA;
        }
    }
    a.nseg = B * L;

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
    int rc;
    if (lse) {
        const size_t n = rows * a.Npad;
        convert_lse_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(lse, N, a.Npad, rows, a.lse2);
        rc = check_launch("convert_lse_kernel");
    } else {
        rc = s->head_dim == 128 ? launch_pass<1, 128>(mq, mk, a, sms, st) : launch_pass<1, 64>(mq, mk, a, sms, st);
    }
    if (rc != PKV_OK) return rc;
    rc = s->head_dim == 128 ? launch_pass<2, 128>(mq, mk, a, sms, st) : launch_pass<2, 64>(mq, mk, a, sms, st);
    if (rc != PKV_OK) return rc;
    return launch_head_mean(a.partial, H, N, (size_t)B * L * N, scores, a.abort_word, st);
}

}  // namespace pkv

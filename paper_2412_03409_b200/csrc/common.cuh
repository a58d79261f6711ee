// Shared host/device helpers of the PrefixKV CUDA library (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "prefixkv.h"

namespace pkv {

constexpr int kMaxPromptLen = 16384;
constexpr size_t kWsAlign = 256;

// Host-side record of the last CUDA error (thread local).
void set_cuda_error(cudaError_t e, const char *where);
void set_error_text(const char *text);
int check_launch(const char *where);
// Raises a kernel's dynamic shared-memory limit once per device.
int ensure_dynamic_smem(const void *func, int bytes, bool *done_per_device);

inline bool shape_ok(const pkv_shape *s)
{
    return s && s->batch > 0 && s->layers > 0 && s->heads > 0 && s->prompt_len > 0 &&
           s->head_dim > 0;
}
inline bool shape_supported(const pkv_shape *s)
{
    if (s->dtype != PKV_F32 && s->dtype != PKV_BF16) return false;
    if (s->head_dim != 64 && s->head_dim != 128) return false;
    if (s->prompt_len > kMaxPromptLen) return false;
    size_t esz = s->dtype == PKV_F32 ? 4 : 2;
    if ((size_t)s->heads * s->head_dim * esz % 16 != 0) return false;
    return true;
}
inline size_t esize(const pkv_shape *s) { return s->dtype == PKV_F32 ? 4 : 2; }
inline bool aligned(const void *p, size_t a) { return ((uintptr_t)p % a) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Launch as a programmatic dependent of the kernel before it in the stream: the grid may be set
// up while that kernel drains; the kernel's own griddepcontrol.wait holds it until the earlier
// kernel has completed and its writes are visible.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                    cudaStream_t st, Args... args)
{
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
// In a kernel launched that way: wait for the earlier kernel, then let the next one be set up.
__device__ __forceinline__ void dependent_entry()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Raise a sample's status word from PKV_DEV_OK; the first condition wins.
__device__ __forceinline__ void raise_status(int32_t *dev_status, int b, int code)
{
    if (dev_status) atomicCAS(dev_status + b, (int)PKV_DEV_OK, code);
}

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_float(float x);
template <> __device__ __forceinline__ float from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x)
{
    return __float2bfloat16_rn(x);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

}  // namespace pkv

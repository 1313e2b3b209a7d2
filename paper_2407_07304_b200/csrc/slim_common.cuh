// Shared device helpers for the SlimAttention kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/slim.h"

namespace slim {

constexpr int kHeadDim = SLIM_HEAD_DIM;       // 128 int8 codes = 128 bytes per cached row
constexpr int kPageTokens = SLIM_PAGE_TOKENS; // rows per page and head
constexpr float kLog2e = 1.4426950408889634f;

// Host-side error plumbing (defined in slim_abi.cu).
int set_cuda_error(cudaError_t e);
#define SLIM_CUDA_TRY(expr)                                       \
    do {                                                          \
        cudaError_t e__ = (expr);                                 \
        if (e__ != cudaSuccess) return slim::set_cuda_error(e__); \
    } while (0)

// Byte / element offsets into the pool (Section 2.2 cache; layout documented in slim.h).
__host__ __device__ inline size_t code_block_offset(int page, int head, int kv, int Hkv)
{
    return ((size_t)((size_t)page * Hkv + head) * 2 + kv) * (size_t)(kPageTokens * kHeadDim);
}
__host__ __device__ inline size_t scale_block_offset(int page, int head, int kv, int Hkv)
{
    return ((size_t)((size_t)page * Hkv + head) * 2 + kv) * (size_t)kPageTokens;
}

// ---------------------------------------------------------------- programmatic dependent launch
// A kernel launched with launch_pdl() may start while the kernel before it in the stream is still
// running (once every block of that kernel has called pdl_launch_dependents() or exited); it must call
// pdl_wait() before it touches anything the earlier kernel writes.  pdl_wait() returns when the
// earlier kernel has completed and its writes are visible; without an earlier kernel it returns at once.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------- small device helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&h);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16)
{
    return __uint_as_float(bits16 << 16);
}

// Largest power of two <= a (a > 0 finite), exponent clamped so that both it and
// its reciprocal are normal floats; the clamp floor for a == 0.
__device__ __forceinline__ float pow2_floor(float a)
{
    int e = (int)((__float_as_uint(a) >> 23) & 0xFF);
    e = max(27, min(227, e));
    return __uint_as_float((uint32_t)e << 23);
}
__device__ __forceinline__ float pow2_recip(float p2)
{
    // p2 = 2^(e-127) with e in [27, 227]  ->  2^(127-e)
    int e = (int)(__float_as_uint(p2) >> 23);
    return __uint_as_float((uint32_t)(254 - e) << 23);
}

// A zero V scale (all-zero row, codes all zero) is replaced by 2^-100 in the decode kernel: the row then
// adds nothing to the numerator and its softmax weight still reaches the denominator.
constexpr float kMinScale = 7.888609052210118e-31f;   // 2^-100

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace slim

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

// ---------------------------------------------------------------- cp.async (16-byte global -> shared)
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;\n" ::: "memory");
}
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// A cached row is 128 bytes = eight 16-byte pieces.  In shared memory piece c of
// row r is stored at piece (c ^ (r & 7)) so that both the row-wise 128-bit reads
// of the score product and the column-wise 32/128-bit reads of the P.V product
// are free of bank conflicts.
__device__ __forceinline__ uint32_t swz_row_piece(int row, int piece)
{
    return (uint32_t)(row * kHeadDim + ((piece ^ (row & 7)) << 4));
}

// ---------------------------------------------------------------- INT8 -> fp16 (exact)
// Hybrid-dtype step of Section 2.2: the codes are converted on the fly, here to
// fp16 (every code in [-128, 127] is exact) for the tensor cores.  A byte u =
// code ^ 0x80 OR-ed into 0x6400 is the fp16 number 1024 + u = 1152 + code; one
// packed subtract of 1152 recovers the code in both halves.
__device__ __forceinline__ uint32_t sub1152(uint32_t h2)
{
    uint32_t r;
    asm("sub.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(h2), "r"(0x64806480u));
    return r;
}
// bytes 0 and 2 of w -> (lo, hi) fp16 pair
__device__ __forceinline__ uint32_t cvt_bytes02(uint32_t w)
{
    return sub1152((w & 0x00FF00FFu) ^ 0x64806480u);
}
// bytes 1 and 3 of w -> (lo, hi) fp16 pair
__device__ __forceinline__ uint32_t cvt_bytes13(uint32_t w)
{
    return sub1152(((w >> 8) & 0x00FF00FFu) ^ 0x64806480u);
}

// ---------------------------------------------------------------- warp-level MMA
// D(16x8, f32) += A(16x16, f16, row) * B(16x8, f16, col)
__device__ __forceinline__ void mma_f16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
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

// log2 and reciprocal of a V scale.  A zero scale (all-zero row, codes all zero) is
// replaced by 2^-100: the row then adds nothing to the numerator and its softmax
// weight still reaches the denominator.
constexpr float kMinScale = 7.888609052210118e-31f;   // 2^-100
__device__ __forceinline__ float log2_scale(float sv)
{
    return __log2f(fmaxf(sv, kMinScale));
}
__device__ __forceinline__ float recip_scale(float sv)
{
    return __frcp_rn(fmaxf(sv, kMinScale));
}

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

// Query A-fragments for the score product.  A thread with quad index t covers
// head dims [32t, 32t+32); k-step j (0..7) contracts dims 32t + 4j + {0,1,2,3},
// paired as (d0, d2) and (d1, d3) to match cvt_bytes02 / cvt_bytes13.
// Each query row is divided by a power of two near its absmax first so that the
// fp16 copy of the bf16 values is exact (no overflow, no loss for values within
// 2^-14 of the row's absmax); the factor is returned in pow2_lo / pow2_hi.
struct QFrag {
    uint32_t a[8][4];
};

// row_lo / row_hi: the 128 bf16 of A-row g and A-row g + 8 (nullptr = zero row).
// With HI == false the upper eight rows are known to be zero and are not touched.
template <bool HI = true>
__device__ __forceinline__ void load_q_frag(QFrag &qf, const __nv_bfloat16 *row_lo, const __nv_bfloat16 *row_hi,
                                            int t, float &pow2_lo, float &pow2_hi)
{
    float x[2][32];
#pragma unroll
    for (int r = 0; r < (HI ? 2 : 1); ++r) {
        const __nv_bfloat16 *row = r ? row_hi : row_lo;
        if (row != nullptr) {
            const uint4 *src = reinterpret_cast<const uint4 *>(row + 32 * t);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 v = __ldg(src + i);
                uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    x[r][i * 8 + 2 * k] = bf16_bits_to_float(w[k] & 0xFFFFu);
                    x[r][i * 8 + 2 * k + 1] = bf16_bits_to_float(w[k] >> 16);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) x[r][i] = 0.f;
        }
    }
    float p2[2] = {1.f, 1.f};
#pragma unroll
    for (int r = 0; r < (HI ? 2 : 1); ++r) {
        float am = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) am = fmaxf(am, fabsf(x[r][i]));
        am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, 1));
        am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, 2));
        p2[r] = pow2_floor(am);
        const float inv = pow2_recip(p2[r]);
#pragma unroll
        for (int i = 0; i < 32; ++i) x[r][i] *= inv;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        qf.a[j][0] = pack_half2(x[0][4 * j + 0], x[0][4 * j + 2]);
        qf.a[j][1] = HI ? pack_half2(x[1][4 * j + 0], x[1][4 * j + 2]) : 0u;
        qf.a[j][2] = pack_half2(x[0][4 * j + 1], x[0][4 * j + 3]);
        qf.a[j][3] = HI ? pack_half2(x[1][4 * j + 1], x[1][4 * j + 3]) : 0u;
    }
    pow2_lo = p2[0];
    pow2_hi = p2[1];
}

// Score product of one 8-token tile: acc(16 x 8) += Q(16 x 128) . K^T, with the
// eight tokens' rows in swizzled shared memory starting at row `row0` (a multiple of 8).
__device__ __forceinline__ void qk_tile(float (&acc)[4], const QFrag &qf, const int8_t *kbuf, int row0, int g, int t)
{
    const int row = row0 + g;
    const uint4 lo = *reinterpret_cast<const uint4 *>(kbuf + swz_row_piece(row, 2 * t));
    const uint4 hi = *reinterpret_cast<const uint4 *>(kbuf + swz_row_piece(row, 2 * t + 1));
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
    for (int j = 0; j < 8; ++j) mma_f16_16816(acc, qf.a[j], cvt_bytes02(w[j]), cvt_bytes13(w[j]));
}

}  // namespace slim

// Quantise-and-append kernel: the write side of the INT8 KV cache (Section 2.2).
//
// The kernel is bound by memory traffic (256 bytes read, 132 written per row), so it is laid out to
// keep many 16-byte loads in flight per thread and to spend few instructions per element:
//
//  * 16 lanes own one row (a lane holds eight consecutive dims: one 16-byte load, one 8-byte store of
//    codes); a block of 256 threads handles 64 consecutive rows, four per half-warp, all loads issued
//    before any arithmetic.
//  * the row quantiser itself (exact round-half-even codes, bit for bit reproducible) is in slim_quant.cuh.
#include "slim_common.cuh"
#include "slim_quant.cuh"

namespace slim {

constexpr int kAppendThreads = 256;
constexpr int kAppendRowsPerGroup = 4;                                       // rows in flight per half-warp
constexpr int kAppendRowsPerBlock = (kAppendThreads / 16) * kAppendRowsPerGroup;   // 64

// grid = (ceil(max_new * Hkv / 64), B, 2 [K, V]); row index = token * Hkv + head within the sequence's new rows.
__global__ void __launch_bounds__(kAppendThreads)
slim_append_kernel(int8_t *__restrict__ codes, float *__restrict__ scales,
                   const int32_t *__restrict__ block_table,
                   const __nv_bfloat16 *__restrict__ k_new, const __nv_bfloat16 *__restrict__ v_new,
                   const int32_t *__restrict__ cu_new, const int32_t *__restrict__ start_pos,
                   int Hkv, int max_pages_per_seq, int num_pages)
{
    pdl_launch_dependents();   // a decode kernel queued behind this one may run its set-up meanwhile
    const int b = blockIdx.y;
    const int kv = blockIdx.z;
    const int hw = threadIdx.x >> 4, l = threadIdx.x & 15;
    const int row0 = __ldg(cu_new + b);
    // 32-bit row arithmetic (the host checks that max_new * Hkv fits): 64-bit divisions would cost more
    // instructions than the quantiser itself
    const int n_rows = (__ldg(cu_new + b + 1) - row0) * Hkv;
    const int first = (int)blockIdx.x * kAppendRowsPerBlock;
    if (first >= n_rows) return;
    const int start = __ldg(start_pos + b);
    const uint4 *src = reinterpret_cast<const uint4 *>((kv ? v_new : k_new) + (size_t)row0 * Hkv * kHeadDim);

    // ---- every load first: the rows' data and the page ids of their destinations
    uint4 raw[kAppendRowsPerGroup];
    int page[kAppendRowsPerGroup], head[kAppendRowsPerGroup], slot[kAppendRowsPerGroup];
#pragma unroll
    for (int i = 0; i < kAppendRowsPerGroup; ++i) {
        const int r = first + i * 16 + hw;     // the block's half-warps cover 16 consecutive rows per step
        page[i] = -1;
        raw[i] = make_uint4(0, 0, 0, 0);
        if (r < n_rows) {
            raw[i] = __ldg(src + (size_t)r * 16 + l);
            const int tok = (int)((unsigned)r / (unsigned)Hkv);
            head[i] = r - tok * Hkv;
            const int pos = start + tok;
            slot[i] = pos & (kPageTokens - 1);
            const int page_idx = pos >> 7;
            if (pos >= 0 && page_idx < max_pages_per_seq) page[i] = __ldg(block_table + (size_t)b * max_pages_per_seq + page_idx);
        }
    }

#pragma unroll
    for (int i = 0; i < kAppendRowsPerGroup; ++i) {
        float scale;
        const uint2 pk = quantize_row16(raw[i], scale);
        if (page[i] >= 0 && page[i] < num_pages) {
            int8_t *dst = codes + code_block_offset(page[i], head[i], kv, Hkv) + (size_t)slot[i] * kHeadDim;
            reinterpret_cast<uint2 *>(dst)[l] = pk;
            if (l == 0) scales[scale_block_offset(page[i], head[i], kv, Hkv) + slot[i]] = scale;
        }
    }
}

int launch_append(const slim_cache_t *c, const void *k_new, const void *v_new, const int32_t *cu_new,
                  const int32_t *start_pos, int B, int max_new, cudaStream_t stream)
{
    const long long rows = (long long)max_new * c->num_kv_heads;
    const long long blocks = (rows + kAppendRowsPerBlock - 1) / kAppendRowsPerBlock;
    if (rows > 0x7FFFFF00LL) return SLIM_ERR_UNSUPPORTED;   // the kernel indexes rows with 32-bit integers
    dim3 grid((unsigned)blocks, (unsigned)B, 2);
    slim_append_kernel<<<grid, kAppendThreads, 0, stream>>>(
        c->codes, c->scales, c->block_table, static_cast<const __nv_bfloat16 *>(k_new),
        static_cast<const __nv_bfloat16 *>(v_new), cu_new, start_pos, c->num_kv_heads, c->max_pages_per_seq,
        c->num_pages);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

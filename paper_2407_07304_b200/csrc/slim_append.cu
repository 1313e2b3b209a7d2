// Quantise-and-append kernel: the write side of the INT8 KV cache (Section 2.2).
#include "slim_common.cuh"

namespace slim {

constexpr int kAppendWarps = 8;

// One warp per (token, kv head) row of K or of V.  Each lane owns four
// consecutive dims: 8-byte load, absmax by shuffles, IEEE divide of the exact
// product 127*x by absmax, round to nearest even, one 4-byte store of codes.
// grid = (ceil(max_new * Hkv / warps), B, 2 [K, V]).
__global__ void __launch_bounds__(kAppendWarps * 32)
slim_append_kernel(int8_t *__restrict__ codes, float *__restrict__ scales,
                   const int32_t *__restrict__ block_table,
                   const __nv_bfloat16 *__restrict__ k_new, const __nv_bfloat16 *__restrict__ v_new,
                   const int32_t *__restrict__ cu_new, const int32_t *__restrict__ start_pos,
                   int Hkv, int max_pages_per_seq, int num_pages)
{
    const int b = blockIdx.y;
    const int kv = blockIdx.z;
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * kAppendWarps + (threadIdx.x >> 5);   // row among this sequence's new rows
    const int row0 = cu_new[b];
    const int n_new = cu_new[b + 1] - row0;
    const int tok = r / Hkv;
    const int head = r - tok * Hkv;
    if (tok >= n_new) return;

    const int pos = start_pos[b] + tok;
    const int page_idx = pos >> 7;
    if (pos < 0 || page_idx >= max_pages_per_seq) return;
    const int page = block_table[(size_t)b * max_pages_per_seq + page_idx];
    if (page < 0 || page >= num_pages) return;
    const int slot = pos & (kPageTokens - 1);

    const __nv_bfloat16 *src = (kv ? v_new : k_new) + ((size_t)(row0 + tok) * Hkv + head) * kHeadDim;
    const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(src) + lane);
    float x[4];
    x[0] = bf16_bits_to_float(raw.x & 0xFFFFu);
    x[1] = bf16_bits_to_float(raw.x >> 16);
    x[2] = bf16_bits_to_float(raw.y & 0xFFFFu);
    x[3] = bf16_bits_to_float(raw.y >> 16);
    float amax = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
    amax = warp_max(amax);

    uint32_t packed = 0;
    if (amax > 0.f) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            // 127*x is exact in fp32 for a bf16 x; the quotient is correctly rounded.
            int c = __float2int_rn(__fdiv_rn(127.f * x[i], amax));
            c = max(-127, min(127, c));
            packed |= ((uint32_t)c & 0xFFu) << (8 * i);
        }
    }
    int8_t *dst = codes + code_block_offset(page, head, kv, Hkv) + (size_t)slot * kHeadDim;
    reinterpret_cast<uint32_t *>(dst)[lane] = packed;
    if (lane == 0)
        scales[scale_block_offset(page, head, kv, Hkv) + slot] = (amax > 0.f) ? __fdiv_rn(amax, 127.f) : 0.f;
}

int launch_append(const slim_cache_t *c, const void *k_new, const void *v_new, const int32_t *cu_new,
                  const int32_t *start_pos, int B, int max_new, cudaStream_t stream)
{
    const long long rows = (long long)max_new * c->num_kv_heads;
    dim3 grid((unsigned)((rows + kAppendWarps - 1) / kAppendWarps), (unsigned)B, 2);
    slim_append_kernel<<<grid, kAppendWarps * 32, 0, stream>>>(
        c->codes, c->scales, c->block_table, static_cast<const __nv_bfloat16 *>(k_new),
        static_cast<const __nv_bfloat16 *>(v_new), cu_new, start_pos, c->num_kv_heads, c->max_pages_per_seq,
        c->num_pages);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

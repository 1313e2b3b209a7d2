// Quantise-and-append kernel: the write side of the INT8 KV cache (Section 2.2).
//
// The kernel is bound by memory traffic (256 bytes read, 132 written per row), so it is laid out to
// keep many 16-byte loads in flight per thread and to spend few instructions per element:
//
//  * 16 lanes own one row (a lane holds eight consecutive dims: one 16-byte load, one 8-byte store of
//    codes); a block of 256 threads handles 64 consecutive rows, four per half-warp, all loads issued
//    before any arithmetic.
//  * code = round_half_even(127 x / amax) on the exact ratio.  The fast path multiplies by the
//    correctly rounded 127 / amax and rounds with the 1.5 * 2^23 trick; the product is within 2^-16 of
//    the exact ratio, so whenever it lies further than 2^-10 from a rounding tie the result is the
//    exact one.  Elements nearer to a tie (0.5 % of them, most of them exact ties of the coarse bf16
//    grid) are redone with the IEEE division of the exact product 127 x by amax, which decides the
//    tie correctly.  Codes and scales are therefore reproducible bit for bit.
#include "slim_common.cuh"

namespace slim {

constexpr int kAppendThreads = 256;
constexpr int kAppendRowsPerGroup = 4;                                       // rows in flight per half-warp
constexpr int kAppendRowsPerBlock = (kAppendThreads / 16) * kAppendRowsPerGroup;   // 64
constexpr float kRoundMagic = 12582912.f;                                    // 1.5 * 2^23

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
    const long long n_rows = (long long)(__ldg(cu_new + b + 1) - row0) * Hkv;
    const long long first = (long long)blockIdx.x * kAppendRowsPerBlock;
    if (first >= n_rows) return;
    const int start = __ldg(start_pos + b);
    const uint4 *src = reinterpret_cast<const uint4 *>((kv ? v_new : k_new) + (size_t)row0 * Hkv * kHeadDim);

    // ---- every load first: the rows' data and the page ids of their destinations
    uint4 raw[kAppendRowsPerGroup];
    int page[kAppendRowsPerGroup], head[kAppendRowsPerGroup], slot[kAppendRowsPerGroup];
#pragma unroll
    for (int i = 0; i < kAppendRowsPerGroup; ++i) {
        const long long r = first + i * 16 + hw;     // the block's half-warps cover 16 consecutive rows per step
        page[i] = -1;
        raw[i] = make_uint4(0, 0, 0, 0);
        if (r < n_rows) {
            raw[i] = __ldg(src + r * 16 + l);
            const int tok = (int)(r / Hkv);
            head[i] = (int)(r - (long long)tok * Hkv);
            const int pos = start + tok;
            slot[i] = pos & (kPageTokens - 1);
            const int page_idx = pos >> 7;
            if (pos >= 0 && page_idx < max_pages_per_seq) page[i] = __ldg(block_table + (size_t)b * max_pages_per_seq + page_idx);
        }
    }

#pragma unroll
    for (int i = 0; i < kAppendRowsPerGroup; ++i) {
        const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
        float x[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            x[2 * k] = __uint_as_float(w[k] << 16);
            x[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
        float amax = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) amax = fmaxf(amax, fabsf(x[k]));
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));   // within the 16 lanes

        uint32_t tb[8];   // low byte = the code in two's complement
        if (amax > 0.f) {
            const float inv = __fdiv_rn(127.f, amax);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float q = x[k] * inv;
                float t = q + kRoundMagic;
                const float d = fabsf(q - (t - kRoundMagic));
                if (d > 0.5f - 0x1p-10f) {
                    // near a rounding tie: 127 * x is exact in fp32 for a bf16 x, the quotient is correctly rounded
                    int c = __float2int_rn(__fdiv_rn(127.f * x[k], amax));
                    c = max(-127, min(127, c));
                    t = __int_as_float(0x4B400000 + c);
                }
                tb[k] = __float_as_uint(t);
            }
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) tb[k] = 0u;
        }
        if (page[i] >= 0 && page[i] < num_pages) {
            uint2 pk;
            pk.x = __byte_perm(__byte_perm(tb[0], tb[1], 0x0040), __byte_perm(tb[2], tb[3], 0x0040), 0x5410);
            pk.y = __byte_perm(__byte_perm(tb[4], tb[5], 0x0040), __byte_perm(tb[6], tb[7], 0x0040), 0x5410);
            int8_t *dst = codes + code_block_offset(page[i], head[i], kv, Hkv) + (size_t)slot[i] * kHeadDim;
            reinterpret_cast<uint2 *>(dst)[l] = pk;
            if (l == 0)
                scales[scale_block_offset(page[i], head[i], kv, Hkv) + slot[i]] = (amax > 0.f) ? __fdiv_rn(amax, 127.f) : 0.f;
        }
    }
}

int launch_append(const slim_cache_t *c, const void *k_new, const void *v_new, const int32_t *cu_new,
                  const int32_t *start_pos, int B, int max_new, cudaStream_t stream)
{
    const long long rows = (long long)max_new * c->num_kv_heads;
    const long long blocks = (rows + kAppendRowsPerBlock - 1) / kAppendRowsPerBlock;
    if (blocks > 0x7FFFFFFFLL) return SLIM_ERR_UNSUPPORTED;
    dim3 grid((unsigned)blocks, (unsigned)B, 2);
    slim_append_kernel<<<grid, kAppendThreads, 0, stream>>>(
        c->codes, c->scales, c->block_table, static_cast<const __nv_bfloat16 *>(k_new),
        static_cast<const __nv_bfloat16 *>(v_new), cu_new, start_pos, c->num_kv_heads, c->max_pages_per_seq,
        c->num_pages);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

// Quantise-and-append kernel: the write side of the INT8 KV cache (Section 2.2).
//
// The kernel is bound by memory traffic (256 bytes read, 132 written per row), so it spends few instructions
// per element and keeps the occupancy an HBM stream needs:
//
//  * 16 / NV lanes own one row (a lane holds NV pieces of eight consecutive dims: a 16-byte load and an
//    8-byte store of codes each), so the per-row work - the shuffle reduction of the maximum, the reciprocal,
//    the scale, token / head / page arithmetic - is shared by 8 NV values per lane.  NV = 4 and one row in
//    flight per group of lanes measured fastest (33 registers, seven blocks of 256 threads per SM); more rows
//    in flight, or 2 / 8 / 16 lanes per row, were 4 to 35 us slower on an 8192-token append.
//  * the row quantiser itself (exact round-half-even codes, bit for bit reproducible) is in slim_quant.cuh.
#include "slim_common.cuh"
#include "slim_quant.cuh"

namespace slim {

constexpr int kAppendNV = 4;               // 16-byte loads per lane and row: four lanes own a row
constexpr int kAppendThreads = 256;
constexpr int kAppendRowsPerGroup = 1;     // rows in flight per group of lanes

// NV = 16-byte loads per lane and row: 16 / NV lanes own a row.
// grid = (ceil(max_new * Hkv / rows per block), B, 2 [K, V]); row index = token * Hkv + head within the
// sequence's new rows.  step_tok / step_head = quotient and remainder of the block's group count by Hkv.
// The first new token of sequence b goes to position start_pos[b], or, without start_pos, to len_after[b] minus the
// sequence's new tokens (the caller states the lengths the sequences have after the append).
template <int NV>
__global__ void __launch_bounds__(kAppendThreads)
slim_append_kernel(int8_t *__restrict__ codes, float *__restrict__ scales,
                   const int32_t *__restrict__ block_table,
                   const __nv_bfloat16 *__restrict__ k_new, const __nv_bfloat16 *__restrict__ v_new,
                   const int32_t *__restrict__ cu_new, const int32_t *__restrict__ start_pos,
                   const int32_t *__restrict__ len_after, int Hkv, int max_pages_per_seq, int num_pages, int step_tok, int step_head)
{
    constexpr int kLanes = 16 / NV;                       // lanes per row
    constexpr int kGroups = kAppendThreads / kLanes;      // rows the block handles per step
    constexpr int kRowsPerBlock = kGroups * kAppendRowsPerGroup;
    pdl_launch_dependents();   // a decode kernel queued behind this one may run its set-up meanwhile
    const int b = blockIdx.y;
    const int kv = blockIdx.z;
    const int g = threadIdx.x / kLanes, l = threadIdx.x % kLanes;
    const int row0 = __ldg(cu_new + b);
    // 32-bit row arithmetic (the host checks that max_new * Hkv fits): 64-bit divisions would cost more
    // instructions than the quantiser itself
    const int n_rows = (__ldg(cu_new + b + 1) - row0) * Hkv;
    const int first = (int)blockIdx.x * kRowsPerBlock;
    if (first >= n_rows) return;
    const int start = (start_pos != nullptr) ? __ldg(start_pos + b) : __ldg(len_after + b) - (__ldg(cu_new + b + 1) - row0);
    const uint4 *src = reinterpret_cast<const uint4 *>((kv ? v_new : k_new) + (size_t)row0 * Hkv * kHeadDim);

    // ---- every load first: the rows' data and the page ids of their destinations.  One division per thread:
    // the rows of a thread are kGroups apart, so token and head advance by fixed steps.
    uint4 raw[kAppendRowsPerGroup][NV];
    int page[kAppendRowsPerGroup], head[kAppendRowsPerGroup], slot[kAppendRowsPerGroup];
    int tok = (int)((unsigned)(first + g) / (unsigned)Hkv);
    int hd = first + g - tok * Hkv;
#pragma unroll
    for (int i = 0; i < kAppendRowsPerGroup; ++i) {
        const int r = first + i * kGroups + g;     // the block's groups cover kGroups consecutive rows per step
        page[i] = -1;
#pragma unroll
        for (int v = 0; v < NV; ++v) raw[i][v] = make_uint4(0, 0, 0, 0);
        if (r < n_rows) {
#pragma unroll
            for (int v = 0; v < NV; ++v) raw[i][v] = __ldg(src + (size_t)r * 16 + v * kLanes + l);
            head[i] = hd;
            const int pos = start + tok;
            slot[i] = pos & (kPageTokens - 1);
            const int page_idx = pos >> 7;
            if (pos >= 0 && page_idx < max_pages_per_seq) page[i] = __ldg(block_table + (size_t)b * max_pages_per_seq + page_idx);
        }
        tok += step_tok;
        hd += step_head;
        if (hd >= Hkv) { hd -= Hkv; ++tok; }
    }

#pragma unroll
    for (int i = 0; i < kAppendRowsPerGroup; ++i) {
        float scale;
        uint2 pk[NV];
        quantize_row<NV>(raw[i], pk, scale);
        if (page[i] >= 0 && page[i] < num_pages) {
            int8_t *dst = codes + code_block_offset(page[i], head[i], kv, Hkv) + (size_t)slot[i] * kHeadDim;
#pragma unroll
            for (int v = 0; v < NV; ++v) reinterpret_cast<uint2 *>(dst)[v * kLanes + l] = pk[v];
            if (l == 0) scales[scale_block_offset(page[i], head[i], kv, Hkv) + slot[i]] = scale;
        }
    }
}

int launch_append(const slim_cache_t *c, const void *k_new, const void *v_new, const int32_t *cu_new,
                  const int32_t *start_pos, int B, int max_new, cudaStream_t stream, const int32_t *len_after)
{
    constexpr int NV = kAppendNV;
    constexpr int kGroups = kAppendThreads / (16 / NV), kRowsPerBlock = kGroups * kAppendRowsPerGroup;
    const long long rows = (long long)max_new * c->num_kv_heads;
    const long long blocks = (rows + kRowsPerBlock - 1) / kRowsPerBlock;
    if (rows > 0x7FFFFF00LL) return SLIM_ERR_UNSUPPORTED;   // the kernel indexes rows with 32-bit integers
    dim3 grid((unsigned)blocks, (unsigned)B, 2);
    slim_append_kernel<NV><<<grid, kAppendThreads, 0, stream>>>(
        c->codes, c->scales, c->block_table, static_cast<const __nv_bfloat16 *>(k_new),
        static_cast<const __nv_bfloat16 *>(v_new), cu_new, start_pos, len_after, c->num_kv_heads, c->max_pages_per_seq,
        c->num_pages, kGroups / c->num_kv_heads, kGroups % c->num_kv_heads);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

// Decode attention over the INT8 KV cache: host-side glue of the two passes and the merge kernel.
//
// The next-token phase is a matrix-vector product bound by memory bandwidth (Section 2.2, Eq. 1: every
// cached byte is read once per generated token).  The key range of every (sequence, kv head) is cut
// into 256-token chunks; the split pass (slim_decode_stream.cu) turns each chunk into a partial result
// (m, l, O[128]) per query head, in SlimAttention order inside the chunk (Section 2.1: all scores, one
// softmax, then .V); the merge pass below combines a row's partials by the log-sum-exp identity.
#include <algorithm>
#include <mutex>

#include "slim_common.cuh"
#include "slim_decode_params.cuh"

namespace slim {

constexpr int kChunkTok = 256;   // tokens per partial result (two pages)
static_assert(kDecodeHeaderBytes == SLIM_WORKSPACE_HEADER_BYTES, "the header size promised in slim.h");

// Partials of a row of `len` cached tokens (never more than cap_tokens): one per 256-token chunk of the
// tokens before the last one, then the last token's own.
__device__ __forceinline__ int merge_row_partials(int len, int cap_tokens)
{
    const int L = min(max(len, 0), cap_tokens);
    return (L == 0) ? 0 : (L - 1 + kChunkTok - 1) / kChunkTok + 1;
}

// Second pass: log-sum-exp merge of a row's chunk partials,
//   M = max m_c;  l = sum l_c 2^(m_c - M);  o = sum O_c 2^(m_c - M) / l.
// One block per (sequence, query head) row: GROUPS groups of 128 threads (thread = head dim), group g takes
// the chunks c = g mod GROUPS, so that a long sequence's hundreds of chunks are read with many independent
// loads in flight (four groups); short rows use one group.  The chunk weights go through shared memory 128
// at a time.
template <int kMergeGroups>
__global__ void __launch_bounds__(kMergeGroups * kHeadDim)
slim_decode_merge_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                         const int32_t *__restrict__ kv_len, __nv_bfloat16 *__restrict__ out, float *__restrict__ raw,
                         int B, int Hq, int n_slots, int cap_tokens)
{
    constexpr int kMergeThreads = kMergeGroups * kHeadDim;
    __shared__ float w_s[kHeadDim];
    __shared__ float red[kMergeThreads / 32];
    __shared__ float acc_s[kMergeGroups][kHeadDim];
    const int row = blockIdx.x;            // b * Hq + h
    const int tid = threadIdx.x, d = tid & (kHeadDim - 1), g = tid >> 7;
    pdl_wait();   // the split pass before this kernel must have finished writing the partials
    const int b = row / Hq;
    const int len = kv_len[b];
    const int nc = merge_row_partials(len, cap_tokens);
    const float2 *ml = reinterpret_cast<const float2 *>(part_ml) + (size_t)row * n_slots;
    const float *po = part_o + (size_t)row * n_slots * kHeadDim;
    // ---- the row's maximum
    float M = -INFINITY;
    for (int c = tid; c < nc; c += kMergeThreads) M = fmaxf(M, ml[c].x);
    M = warp_max(M);
    if ((tid & 31) == 0) red[tid >> 5] = M;
    __syncthreads();
    M = red[0];
#pragma unroll
    for (int i = 1; i < kMergeThreads / 32; ++i) M = fmaxf(M, red[i]);
    // ---- weighted sums, 128 chunks per round
    float acc = 0.f, lsum = 0.f;
    for (int c0 = 0; c0 < nc; c0 += kHeadDim) {
        const int n = min(kHeadDim, nc - c0);
        __syncthreads();                   // the previous round's weights (and the maxima) have been used
        if (tid < n) {
            const float2 v = ml[c0 + tid];
            const float w = exp2f(v.x - M);
            w_s[tid] = w;
            lsum = fmaf(v.y, w, lsum);
        }
        __syncthreads();
        const float *src = po + (size_t)c0 * kHeadDim + d;
        int c = g;
        for (; c + 3 * kMergeGroups < n; c += 4 * kMergeGroups) {
            const float v0 = src[(size_t)c * kHeadDim], v1 = src[(size_t)(c + kMergeGroups) * kHeadDim];
            const float v2 = src[(size_t)(c + 2 * kMergeGroups) * kHeadDim], v3 = src[(size_t)(c + 3 * kMergeGroups) * kHeadDim];
            acc = fmaf(v0, w_s[c], acc);
            acc = fmaf(v1, w_s[c + kMergeGroups], acc);
            acc = fmaf(v2, w_s[c + 2 * kMergeGroups], acc);
            acc = fmaf(v3, w_s[c + 3 * kMergeGroups], acc);
        }
        for (; c < n; c += kMergeGroups) acc = fmaf(src[(size_t)c * kHeadDim], w_s[c], acc);
    }
    // ---- combine the four groups and the denominators (only the first 128 threads hold a share of lsum)
    acc_s[g][d] = acc;
    lsum = warp_sum(lsum);
    __syncthreads();                       // red is free again (every thread has read the maxima)
    if ((tid & 31) == 0) red[tid >> 5] = lsum;
    __syncthreads();
    if (g == 0) {
        const float l = (red[0] + red[1]) + (red[2] + red[3]);   // the first four warps hold the shares
        float o = acc_s[0][d];
#pragma unroll
        for (int i = 1; i < kMergeGroups; ++i) o += acc_s[i][d];
        if (raw != nullptr) {
            // the row's merged partial instead of its normalised result (the keys are split over several devices)
            float *dst = raw + (size_t)row * SLIM_PARTIAL_FLOATS;
            dst[d] = (nc > 0) ? o : 0.f;
            if (d == 0) dst[kHeadDim] = (nc > 0) ? M : -INFINITY, dst[kHeadDim + 1] = (nc > 0) ? l : 0.f;
            return;
        }
        const float inv = (nc > 0 && l > 0.f) ? 1.f / l : 0.f;
        out[(size_t)row * kHeadDim + d] = __float2bfloat16_rn(o * inv);
    }
}

// A row's merged partial (what slim_attn_decode_partial returns): O relative to M, then M and l; a lane owns four dims.
__device__ __forceinline__ void store_raw_partial(float *raw, int row, int lane, float4 o, float M, float l)
{
    float *dst = raw + (size_t)row * SLIM_PARTIAL_FLOATS;
    reinterpret_cast<float4 *>(dst)[lane] = o;
    if (lane == 0) *reinterpret_cast<float2 *>(dst + kHeadDim) = make_float2(M, l);
}

// A 16-byte load past the L1 cache that the compiler keeps where it is written (the merge kernels request a
// row's partials before the values that decide which of them count have arrived).
__device__ __forceinline__ float4 ld_cg_now(const float4 *ptr)
{
    float4 v;
    asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr) : "memory");
    return v;
}

// The same merge for rows of fewer than 32 chunks: one warp per (sequence, query head) row, a lane owns four head
// dims, lane c owns chunk c's (m, l).  Once the row's length has arrived, the (m, l) pairs and the first sixteen
// partial outputs of the row are requested together, so a row costs two round trips to memory instead of one per
// step of the reduction.  (Asking for the sixteen slots before the length is known, as the block-per-row kernel below
// does, read half as much again on ragged batches and was 0.5 us slower on the 64 / 8-head workload.)
constexpr int kMergeWarpBatch = 16;
constexpr int kMergeWarpsPerBlock = 8;
__global__ void __launch_bounds__(kMergeWarpsPerBlock * 32)
slim_decode_merge_warp_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                              const int32_t *__restrict__ kv_len, __nv_bfloat16 *__restrict__ out, float *__restrict__ raw,
                              int B, int Hq, int n_slots, int cap_tokens)
{
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kMergeWarpsPerBlock + (threadIdx.x >> 5);   // b * Hq + h
    pdl_wait();   // the split pass before this kernel must have finished writing the partials
    if (row >= B * Hq) return;
    const int len = __ldg(kv_len + row / Hq);
    const float2 *ml = reinterpret_cast<const float2 *>(part_ml) + (size_t)row * n_slots;
    const float4 *po = reinterpret_cast<const float4 *>(part_o + (size_t)row * n_slots * kHeadDim) + lane;
    const int nc = merge_row_partials(len, cap_tokens);
    float4 o[kMergeWarpBatch];
#pragma unroll
    for (int u = 0; u < kMergeWarpBatch; ++u)
        o[u] = (u < nc) ? __ldcg(po + (size_t)u * (kHeadDim / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    float2 v = (lane < nc) ? __ldcg(ml + lane) : make_float2(-INFINITY, 0.f);
    if (lane >= nc) v = make_float2(-INFINITY, 0.f);
    const float M = warp_max(v.x);
    const float w = (lane < nc) ? exp2f(v.x - M) : 0.f;
    const float l = warp_sum(v.y * w);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c0 = 0; c0 < nc; c0 += kMergeWarpBatch) {
        if (c0 > 0) {
#pragma unroll
            for (int u = 0; u < kMergeWarpBatch; ++u)
                o[u] = (c0 + u < nc) ? __ldcg(po + (size_t)(c0 + u) * (kHeadDim / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kMergeWarpBatch; ++u) {
            const float wj = __shfl_sync(0xffffffffu, w, (c0 + u) & 31);
            if (c0 + u < nc) {
                acc.x = fmaf(o[u].x, wj, acc.x);
                acc.y = fmaf(o[u].y, wj, acc.y);
                acc.z = fmaf(o[u].z, wj, acc.z);
                acc.w = fmaf(o[u].w, wj, acc.w);
            }
        }
    }
    if (raw != nullptr) {
        store_raw_partial(raw, row, lane, nc > 0 ? acc : make_float4(0.f, 0.f, 0.f, 0.f), nc > 0 ? M : -INFINITY, nc > 0 ? l : 0.f);
        return;
    }
    const float inv = (nc > 0 && l > 0.f) ? 1.f / l : 0.f;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t *>(&lo);
    packed.y = *reinterpret_cast<uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(out + (size_t)row * kHeadDim + lane * 4) = packed;
}

// Rows of 32 to 16 * kWarps chunks: one block per row, warp w owns the sixteen chunk slots [16 w, 16 w + 16) and
// merges them as the kernel above does - all of its partials requested at once, before the row's length is known -
// into (M_w, l_w, o_w); the warps' results are then merged by the same identity through shared memory.
template <int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1)
slim_decode_merge_block_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                               const int32_t *__restrict__ kv_len, __nv_bfloat16 *__restrict__ out, float *__restrict__ raw,
                               int B, int Hq, int n_slots, int cap_tokens)
{
    __shared__ float4 acc_s[kWarps][32];
    __shared__ float m_s[kWarps], l_s[kWarps];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int row = blockIdx.x;   // b * Hq + h
    pdl_wait();   // the split pass before this kernel must have finished writing the partials
    const int len = __ldg(kv_len + row / Hq);
    const int c_base = w * kMergeWarpBatch;
    const float2 *ml = reinterpret_cast<const float2 *>(part_ml) + (size_t)row * n_slots;
    const float4 *po = reinterpret_cast<const float4 *>(part_o + (size_t)row * n_slots * kHeadDim) + lane;
    float4 o[kMergeWarpBatch];
#pragma unroll
    for (int u = 0; u < kMergeWarpBatch; ++u)
        o[u] = ld_cg_now(po + (size_t)min(c_base + u, n_slots - 1) * (kHeadDim / 4));   // n_slots >= 32 here; slots past nc are not used
    float2 v = (lane < kMergeWarpBatch && c_base + lane < n_slots) ? __ldcg(ml + c_base + lane) : make_float2(-INFINITY, 0.f);
    const int nc = merge_row_partials(len, cap_tokens);
    const bool mine = lane < kMergeWarpBatch && c_base + lane < nc;
    if (!mine) v = make_float2(-INFINITY, 0.f);
    const float Mw = warp_max(v.x);
    const float wgt = mine ? exp2f(v.x - Mw) : 0.f;
    const float lw = warp_sum(v.y * wgt);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < kMergeWarpBatch; ++u) {
        const float wj = __shfl_sync(0xffffffffu, wgt, u);
        if (c_base + u < nc) {   // a slot past the row's last chunk may hold anything, a NaN included
            acc.x = fmaf(o[u].x, wj, acc.x);
            acc.y = fmaf(o[u].y, wj, acc.y);
            acc.z = fmaf(o[u].z, wj, acc.z);
            acc.w = fmaf(o[u].w, wj, acc.w);
        }
    }
    acc_s[w][lane] = acc;
    if (lane == 0) {
        m_s[w] = Mw;   // minus infinity for a warp whose slots lie past the row's last chunk
        l_s[w] = lw;
    }
    __syncthreads();
    if (w == 0) {
        float M = -INFINITY;
#pragma unroll
        for (int i = 0; i < kWarps; ++i) M = fmaxf(M, m_s[i]);
        float l = 0.f;
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < kWarps; ++i) {
            const float f = (m_s[i] == -INFINITY) ? 0.f : exp2f(m_s[i] - M);
            const float4 a = acc_s[i][lane];
            l = fmaf(l_s[i], f, l);
            r.x = fmaf(a.x, f, r.x);
            r.y = fmaf(a.y, f, r.y);
            r.z = fmaf(a.z, f, r.z);
            r.w = fmaf(a.w, f, r.w);
        }
        if (raw != nullptr) {
            store_raw_partial(raw, row, lane, nc > 0 ? r : make_float4(0.f, 0.f, 0.f, 0.f), nc > 0 ? M : -INFINITY, nc > 0 ? l : 0.f);
            return;
        }
        const float inv = (nc > 0 && l > 0.f) ? 1.f / l : 0.f;
        __nv_bfloat162 lo = __floats2bfloat162_rn(r.x * inv, r.y * inv), hi = __floats2bfloat162_rn(r.z * inv, r.w * inv);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t *>(&lo);
        packed.y = *reinterpret_cast<uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(out + (size_t)row * kHeadDim + lane * 4) = packed;
    }
}

// ---------------------------------------------------------------- host side
size_t decode_workspace_bytes(int B, int Hq, int Hkv, int max_kv)
{
    (void)Hkv;
    const size_t slots = (size_t)(max_kv + kChunkTok - 1) / kChunkTok + 1;   // a row's chunks and its last token
    return kDecodeHeaderBytes + (size_t)B * Hq * slots * (kHeadDim + 2) * sizeof(float);
}

static DecodeParams make_params(const slim_cache_t *c, const void *q, const int32_t *kv_len, int B, int max_kv,
                                int Hq, float sm_scale, void *workspace, int &C)
{
    const int Hkv = c->num_kv_heads;
    C = kChunkTok;
    DecodeParams p;
    p.codes = c->codes;
    p.scales = c->scales;
    p.block_table = c->block_table;
    p.kv_len = kv_len;
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.G = Hq / Hkv;
    p.max_pages_per_seq = c->max_pages_per_seq;
    p.num_pages = c->num_pages;
    p.n_chunks = (max_kv + C - 1) / C;
    p.n_slots = p.n_chunks + 1;
    p.scale_log2e = sm_scale * kLog2e;
    p.status = static_cast<int *>(workspace);
    p.part_o = reinterpret_cast<float *>(static_cast<char *>(workspace) + kDecodeHeaderBytes);
    p.part_ml = p.part_o + (size_t)B * Hq * p.n_slots * kHeadDim;
    p.k_new = p.v_new = nullptr;
    p.out = nullptr;
    p.counters = nullptr;
    return p;
}

int launch_decode_split(const slim_cache_t *c, const void *q, const void *k_new, const void *v_new, const int32_t *kv_len,
                        int B, int max_kv, int Hq, float sm_scale, void *workspace, cudaStream_t stream)
{
    int C;
    DecodeParams p = make_params(c, q, kv_len, B, max_kv, Hq, sm_scale, workspace, C);
    if (p.n_chunks == 0) return SLIM_OK;
    p.k_new = static_cast<const __nv_bfloat16 *>(k_new);
    p.v_new = static_cast<const __nv_bfloat16 *>(v_new);
    return launch_decode_split_stream(c, p, B, stream);
}

int launch_decode_merge(const slim_cache_t *c, void *out, const int32_t *kv_len, int B, int max_kv, int Hq,
                        const void *workspace, cudaStream_t stream, float *raw = nullptr);

// Decode attention.  With k_new / v_new the split kernel first quantises every sequence's new token into slot
// kv_len - 1 of the cache (the one-call decode step).  Where a (sequence, kv head) has few partials the split
// kernel merges them itself when its blocks finish (one warp per pair); otherwise the merge kernel follows.
constexpr int kInKernelMergeMaxPartials = 32;   // G * chunks of a (sequence, kv head) that one warp merges at the end of a block

int launch_decode(const slim_cache_t *c, const void *q, const void *k_new, const void *v_new, void *out,
                  const int32_t *kv_len, int B, int max_kv, int Hq, float sm_scale, void *workspace, cudaStream_t stream)
{
    int C;
    DecodeParams p = make_params(c, q, kv_len, B, max_kv, Hq, sm_scale, workspace, C);
    if (p.n_chunks == 0) return launch_decode_merge(c, out, kv_len, B, max_kv, Hq, workspace, stream);   // rows of zeros
    p.k_new = static_cast<const __nv_bfloat16 *>(k_new);
    p.v_new = static_cast<const __nv_bfloat16 *>(v_new);
    const bool in_kernel = (long long)B * p.Hkv <= kDecodeCounterRows && p.G * p.n_slots <= kInKernelMergeMaxPartials;
    if (in_kernel) {
        p.out = static_cast<__nv_bfloat16 *>(out);
        p.counters = reinterpret_cast<int *>(static_cast<char *>(workspace) + kDecodeStatusBytes);
    }
    const int rc = launch_decode_split_stream(c, p, B, stream);
    if (rc != SLIM_OK || in_kernel) return rc;
    return launch_decode_merge(c, out, kv_len, B, max_kv, Hq, workspace, stream);
}

int launch_decode_merge(const slim_cache_t *c, void *out, const int32_t *kv_len, int B, int max_kv, int Hq,
                        const void *workspace, cudaStream_t stream, float *raw)
{
    int C;
    const DecodeParams p = make_params(c, nullptr, kv_len, B, max_kv, Hq, 1.f, const_cast<void *>(workspace), C);
    const int rows = B * Hq;
    const int cap = (int)std::min<long long>((long long)c->max_pages_per_seq * kPageTokens, (long long)p.n_chunks * C);
    const float *po = p.part_o, *pm = p.part_ml;
    __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(out);
    if (p.n_slots >= 32 && p.n_slots <= 16 * kMergeWarpBatch) {
        if (p.n_slots <= 4 * kMergeWarpBatch)
            SLIM_CUDA_TRY(launch_pdl(slim_decode_merge_block_kernel<4>, dim3(rows), dim3(128), 0, stream, po, pm, kv_len, o, raw, B, Hq, p.n_slots, cap));
        else if (p.n_slots <= 8 * kMergeWarpBatch)
            SLIM_CUDA_TRY(launch_pdl(slim_decode_merge_block_kernel<8>, dim3(rows), dim3(256), 0, stream, po, pm, kv_len, o, raw, B, Hq, p.n_slots, cap));
        else
            SLIM_CUDA_TRY(launch_pdl(slim_decode_merge_block_kernel<16>, dim3(rows), dim3(512), 0, stream, po, pm, kv_len, o, raw, B, Hq, p.n_slots, cap));
    } else if (p.n_slots >= 32) {
        SLIM_CUDA_TRY(launch_pdl(slim_decode_merge_kernel<4>, dim3(rows), dim3(4 * kHeadDim), 0, stream, po, pm, kv_len, o, raw, B, Hq, p.n_slots, cap));
    } else {
        const int blocks = (rows + kMergeWarpsPerBlock - 1) / kMergeWarpsPerBlock;
        SLIM_CUDA_TRY(launch_pdl(slim_decode_merge_warp_kernel, dim3(blocks), dim3(kMergeWarpsPerBlock * 32), 0, stream, po, pm, kv_len, o, raw, B, Hq,
                                 p.n_slots, cap));
    }
    return SLIM_OK;
}

// Decode attention over a part of every sequence's keys: split pass, then the merge pass leaves each row's merged
// partial (O, M, l) instead of the normalised result.
int launch_decode_partial(const slim_cache_t *c, const void *q, float *partial, const int32_t *kv_len, int B, int max_kv, int Hq,
                          float sm_scale, void *workspace, cudaStream_t stream)
{
    int C;
    DecodeParams p = make_params(c, q, kv_len, B, max_kv, Hq, sm_scale, workspace, C);
    if (p.n_chunks > 0) {
        const int rc = launch_decode_split_stream(c, p, B, stream);
        if (rc != SLIM_OK) return rc;
    }
    return launch_decode_merge(c, nullptr, kv_len, B, max_kv, Hq, workspace, stream, partial);
}

// Final merge over R sets of row partials (one set per device that holds a part of the keys):
//   M = max M_r;  l = sum l_r 2^(M_r - M);  o = sum O_r 2^(M_r - M) / l.   One warp per row, a lane owns four dims.
__global__ void __launch_bounds__(256)
slim_merge_partials_kernel(const float *__restrict__ parts, int R, int rows, __nv_bfloat16 *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    float M = -INFINITY;
    for (int r = 0; r < R; ++r) M = fmaxf(M, __ldg(parts + ((size_t)r * rows + row) * SLIM_PARTIAL_FLOATS + kHeadDim));
    float l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r = 0; r < R; ++r) {
        const float *src = parts + ((size_t)r * rows + row) * SLIM_PARTIAL_FLOATS;
        const float2 ml = __ldg(reinterpret_cast<const float2 *>(src + kHeadDim));
        if (ml.x == -INFINITY) continue;   // a device whose part of this sequence is empty
        const float w = exp2f(ml.x - M);
        const float4 o = __ldg(reinterpret_cast<const float4 *>(src) + lane);
        l = fmaf(ml.y, w, l);
        acc.x = fmaf(o.x, w, acc.x);
        acc.y = fmaf(o.y, w, acc.y);
        acc.z = fmaf(o.z, w, acc.z);
        acc.w = fmaf(o.w, w, acc.w);
    }
    const float inv = (l > 0.f) ? 1.f / l : 0.f;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t *>(&lo);
    packed.y = *reinterpret_cast<uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(out + (size_t)row * kHeadDim + lane * 4) = packed;
}

int launch_merge_partials(const float *parts, int R, int rows, void *out, cudaStream_t stream)
{
    slim_merge_partials_kernel<<<(rows + 7) / 8, 256, 0, stream>>>(parts, R, rows, static_cast<__nv_bfloat16 *>(out));
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

// ---------------------------------------------------------------- decode without a caller-provided workspace
//
// Scratch for slim_attn_decode_static: the split pass's partial results live in this
// file-scope device array instead of a buffer the caller allocates.  Every GPU that loads
// the library carries these bytes until the process exits, so the size is kept modest.
static __device__ __align__(256) unsigned char g_static_decode_scratch[SLIM_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_scratch_mu;               // guards the two tables below (host threads may make their first call together)
void *g_static_scratch_ptr[kMaxDevices];      // device address of the array, per device ordinal
bool g_static_scratch_ready[kMaxDevices];
}  // namespace

// In host code the array's name only stands for the symbol; the address a kernel can use has
// to be asked for, once per device, while that device is current.
static int static_scratch_address(void **ptr)
{
    int dev = -1;
    SLIM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SLIM_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_scratch_mu);
    if (!g_static_scratch_ready[dev]) {
        void *addr = nullptr;
        SLIM_CUDA_TRY(cudaGetSymbolAddress(&addr, g_static_decode_scratch));
        g_static_scratch_ptr[dev] = addr;
        g_static_scratch_ready[dev] = true;
    }
    *ptr = g_static_scratch_ptr[dev];
    return SLIM_OK;
}

extern "C" __attribute__((visibility("default")))
int slim_attn_decode_static(const slim_cache_t *cache, const void *q, void *out, const int32_t *kv_len, int32_t B,
                            int32_t max_kv, int32_t Hq, float sm_scale, void *stream)
{
    using namespace slim;
    if (cache == nullptr || cache->codes == nullptr || cache->scales == nullptr || cache->block_table == nullptr)
        return SLIM_ERR_INVALID_ARG;
    if (cache->num_pages <= 0 || cache->num_kv_heads <= 0 || cache->max_pages_per_seq <= 0) return SLIM_ERR_INVALID_ARG;
    if (cache->page_tokens != SLIM_PAGE_TOKENS || cache->head_dim != SLIM_HEAD_DIM) return SLIM_ERR_UNSUPPORTED;
    if (((uintptr_t)cache->codes & 15) || ((uintptr_t)cache->scales & 15)) return SLIM_ERR_INVALID_ARG;
    if (B < 0 || max_kv < 0 || Hq <= 0) return SLIM_ERR_INVALID_ARG;
    if (Hq % cache->num_kv_heads != 0 || Hq / cache->num_kv_heads > 16) return SLIM_ERR_UNSUPPORTED;
    if (B == 0) return SLIM_OK;
    if (B > 65535 || cache->num_kv_heads > 65535) return SLIM_ERR_UNSUPPORTED;
    if ((long long)max_kv > (long long)cache->max_pages_per_seq * SLIM_PAGE_TOKENS) return SLIM_ERR_INVALID_ARG;
    if (q == nullptr || out == nullptr || kv_len == nullptr) return SLIM_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return SLIM_ERR_INVALID_ARG;
    // the problem must fit the built-in scratch: there is nothing to fall back to
    if (decode_workspace_bytes(B, Hq, cache->num_kv_heads, max_kv) > (size_t)SLIM_STATIC_SCRATCH_BYTES)
        return SLIM_ERR_WORKSPACE;
    void *scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != SLIM_OK) return rc;
    return launch_decode(cache, q, nullptr, nullptr, out, kv_len, B, max_kv, Hq, sm_scale, scratch, (cudaStream_t)stream);
}

// The built-in array's header (status word and merge counters) is out of the caller's reach, so these three calls
// stand in for slim_read_status, a cudaMemset of the header and slim_selftest_timeout on an ordinary workspace.
extern "C" __attribute__((visibility("default")))
int slim_static_status(void *stream)
{
    void *scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != SLIM_OK) return rc;
    return slim_read_status(scratch, stream);
}

extern "C" __attribute__((visibility("default")))
int slim_static_reset(void *stream)
{
    void *scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != SLIM_OK) return rc;
    SLIM_CUDA_TRY(cudaMemsetAsync(scratch, 0, SLIM_WORKSPACE_HEADER_BYTES, (cudaStream_t)stream));
    return SLIM_OK;
}

extern "C" __attribute__((visibility("default")))
int slim_static_selftest_timeout(void *stream)
{
    void *scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != SLIM_OK) return rc;
    return slim_selftest_timeout(scratch, stream);
}

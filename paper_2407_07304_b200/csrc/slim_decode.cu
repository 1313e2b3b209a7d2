// Decode attention over the INT8 KV cache: split kernel + merge kernel.
//
// The next-token phase is a matrix-vector product bound by memory bandwidth
// (Section 2.2, Eq. 1: every cached byte is read once per generated token), so
// the kernel is organised around keeping the whole key range in flight:
// a thread block owns one (sequence, kv head, chunk of keys), asks for its whole
// chunk with 16-byte asynchronous copies at once, and consumes it as it lands.
// Inside a chunk the order is SlimAttention's (Section 2.1): all scores of the
// chunk first, one softmax over them, then the product with V - no running
// rescale.  The G = Hq / Hkv query heads that share the kv head form the rows of
// a 16-row tensor-core tile, so each cached byte is converted and used once for
// all of them.
//
// The V scale of key j is folded into the softmax weight: with
//   s'_j = s_j + log2(scale_v[j]),  m' = max_j s'_j,  P_j = 2^(s'_j - m')
// the output is  o = (sum_j P_j * v_code_j) / (sum_j P_j / scale_v[j]),
// identical to softmax(s) . (v_code * scale_v) because the factor 2^(-m') cancels.
// P_j <= 1 is normalised by the row's largest contribution, which is what makes
// its fp16 copy for the tensor cores safe whatever the spread of the V scales.
#include "slim_common.cuh"

namespace slim {

constexpr int kDecodeThreads = 128;
constexpr int kDecodeWarps = 4;
constexpr int kWarpTok = 64;                              // tokens owned by one warp
constexpr int kChunkTok = kDecodeWarps * kWarpTok;        // tokens per thread block (two pages)

struct DecodeParams {
    const int8_t *codes;
    const float *scales;
    const int32_t *block_table;
    const int32_t *kv_len;
    const __nv_bfloat16 *q;   // [B][Hq][128]
    float *part_o;            // [B][Hq][n_chunks][128] unnormalised partial outputs
    float *part_ml;           // [B][Hq][n_chunks][2]   (max in log2 units, sum)
    int Hq, Hkv, G;
    int max_pages_per_seq, num_pages, n_chunks;
    float scale_log2e;        // sm_scale * log2(e)
};

// Shared memory of one warp: its 64 tokens' K and V rows (swizzled, see swz_row_piece) and
// scales.  After the warp has consumed them the same bytes hold its partial result.
struct __align__(128) WarpBuf {
    int8_t k[kWarpTok * kHeadDim];
    int8_t v[kWarpTok * kHeadDim];
    float ks[kWarpTok];
    float vs[kWarpTok];
};
constexpr int kORowStride = 144;   // floats per partial-output row: four 32-float groups padded to 36

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// ROWS: query heads per kv head, rounded up to 8 or 16 (rows of the 16-row MMA tile in use).
//
// A block owns 256 consecutive tokens of one (sequence, kv head); each of its four warps owns
// 64 of them and works alone: it asks for its K rows, V rows and scales with 16-byte
// asynchronous copies (all in flight at once), then follows the SlimAttention order on its
// slice - all 64 scores, one softmax over them, then the product with V - entirely in
// registers.  The four slices are merged through shared memory and written as one partial.
template <int ROWS>
__global__ void __launch_bounds__(kDecodeThreads)
slim_decode_split_kernel(const DecodeParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int chunk = blockIdx.x, head = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int len = min(p.kv_len[b], p.max_pages_per_seq * kPageTokens);
    const int n_tok = min(kChunkTok, len - chunk * kChunkTok);   // valid tokens of this block
    if (n_tok <= 0) return;
    WarpBuf &wb = reinterpret_cast<WarpBuf *>(smem)[warp];
    const int n_w = max(0, min(kWarpTok, n_tok - warp * kWarpTok));   // valid tokens of this warp
    const int h0 = head * p.G;

    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
    float m_row[2] = {-INFINITY, -INFINITY}, l_row[2] = {0.f, 0.f};

    if (n_w > 0) {
        // ---- ask for everything this warp will read: K rows + both scale vectors, then V rows
        int page = p.block_table[(size_t)b * p.max_pages_per_seq + chunk * 2 + (warp >> 1)];
        page = (page >= 0 && page < p.num_pages) ? page : 0;
        const int slot0 = (warp & 1) * kWarpTok;
        {
            const int r0 = lane >> 3, c = lane & 7;
            // rows r0 + 4*it: (row & 7) alternates between r0 and r0 + 4
            const uint32_t dsw[2] = {(uint32_t)((c ^ r0) << 4), (uint32_t)((c ^ (r0 + 4)) << 4)};
#pragma unroll
            for (int kv = 0; kv < 2; ++kv) {
                const int8_t *src = p.codes + code_block_offset(page, head, kv, p.Hkv) +
                                    (size_t)(slot0 + r0) * kHeadDim + c * 16;
                const uint32_t dst = smem_u32(kv ? wb.v : wb.k) + r0 * kHeadDim;
#pragma unroll
                for (int it = 0; it < 16; ++it)
                    if (r0 + 4 * it < n_w) cp_async16(dst + it * 4 * kHeadDim + dsw[it & 1], src + it * 4 * kHeadDim);
                if (kv == 0) {
                    const int which = lane >> 4, qd = lane & 15;
                    if (qd * 4 < n_w)
                        cp_async16(smem_u32((which ? wb.vs : wb.ks) + qd * 4),
                                   p.scales + scale_block_offset(page, head, which, p.Hkv) + slot0 + qd * 4);
                }
                cp_async_commit();
            }
        }

        // ---- query fragments (rows = the G heads of this kv head), while the copies fly
        const __nv_bfloat16 *qbase = p.q + ((size_t)b * p.Hq + h0) * kHeadDim;
        QFrag qf;
        float pow2_lo, pow2_hi;
        load_q_frag<(ROWS > 8)>(qf, (g < p.G) ? qbase + (size_t)g * kHeadDim : nullptr,
                                (ROWS > 8 && g + 8 < p.G) ? qbase + (size_t)(g + 8) * kHeadDim : nullptr, t,
                                pow2_lo, pow2_hi);
        const float rs[2] = {pow2_lo * p.scale_log2e, pow2_hi * p.scale_log2e};

        // ---- all scores of the slice (log2 units, V scale folded in): s[nt] = tokens 8nt + {2t, 2t+1}
        cp_async_wait<1>();
        __syncwarp();
        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int j = 0; j < 4; ++j) s[nt][j] = 0.f;
            if (nt * 8 < n_w) qk_tile(s[nt], qf, wb.k, nt * 8, g, t);
        }
        float rsv[8][2];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float2 sk = *reinterpret_cast<const float2 *>(wb.ks + nt * 8 + 2 * t);
            const float2 sv = *reinterpret_cast<const float2 *>(wb.vs + nt * 8 + 2 * t);
            const bool v0 = nt * 8 + 2 * t < n_w, v1 = nt * 8 + 2 * t + 1 < n_w;
            const float l0 = log2_scale(sv.x), l1 = log2_scale(sv.y);
            rsv[nt][0] = v0 ? recip_scale(sv.x) : 0.f;
            rsv[nt][1] = v1 ? recip_scale(sv.y) : 0.f;
            s[nt][0] = v0 ? fmaf(s[nt][0], sk.x * rs[0], l0) : -INFINITY;
            s[nt][1] = v1 ? fmaf(s[nt][1], sk.y * rs[0], l1) : -INFINITY;
            if (ROWS > 8) {
                s[nt][2] = v0 ? fmaf(s[nt][2], sk.x * rs[1], l0) : -INFINITY;
                s[nt][3] = v1 ? fmaf(s[nt][3], sk.y * rs[1], l1) : -INFINITY;
            }
            m_row[0] = fmaxf(m_row[0], fmaxf(s[nt][0], s[nt][1]));
            if (ROWS > 8) m_row[1] = fmaxf(m_row[1], fmaxf(s[nt][2], s[nt][3]));
        }
        // ---- one softmax over the slice: P = 2^(s' - m') as fp16 A-fragments, l = sum P / scale_v
        uint32_t pa[4][4];
#pragma unroll
        for (int r = 0; r < (ROWS > 8 ? 2 : 1); ++r) {
            m_row[r] = fmaxf(m_row[r], __shfl_xor_sync(0xffffffffu, m_row[r], 1));
            m_row[r] = fmaxf(m_row[r], __shfl_xor_sync(0xffffffffu, m_row[r], 2));
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float e0 = fast_exp2(s[nt][0] - m_row[0]), e1 = fast_exp2(s[nt][1] - m_row[0]);
            l_row[0] = fmaf(e0, rsv[nt][0], fmaf(e1, rsv[nt][1], l_row[0]));
            pa[nt >> 1][(nt & 1) * 2] = pack_half2(e0, e1);
            if (ROWS > 8) {
                const float e2 = fast_exp2(s[nt][2] - m_row[1]), e3 = fast_exp2(s[nt][3] - m_row[1]);
                l_row[1] = fmaf(e2, rsv[nt][0], fmaf(e3, rsv[nt][1], l_row[1]));
                pa[nt >> 1][(nt & 1) * 2 + 1] = pack_half2(e2, e3);
            } else {
                pa[nt >> 1][(nt & 1) * 2 + 1] = 0u;
            }
        }
#pragma unroll
        for (int r = 0; r < (ROWS > 8 ? 2 : 1); ++r) {
            l_row[r] += __shfl_xor_sync(0xffffffffu, l_row[r], 1);
            l_row[r] += __shfl_xor_sync(0xffffffffu, l_row[r], 2);
        }

        // ---- O = P . V over the slice in steps of 16 tokens; thread (g, t) supplies head dims
        //      16g + [0, 16) of token rows 16ks + {2t, 2t+1, 2t+8, 2t+9}
        cp_async_wait<0>();
        __syncwarp();
        const uint32_t voff0 = (uint32_t)((2 * t) * kHeadDim + ((g ^ (2 * t)) << 4));
        const uint32_t voff1 = (uint32_t)((2 * t + 1) * kHeadDim + ((g ^ (2 * t + 1)) << 4));
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            if (ks * 16 < n_w) {
                // rows past the slice's last token hold stale bytes: any byte converts to a finite
                // fp16 and its P entry is zero, so they add nothing
                const int8_t *vb = wb.v + ks * 16 * kHeadDim;
                const uint4 w0 = *reinterpret_cast<const uint4 *>(vb + voff0);
                const uint4 w1 = *reinterpret_cast<const uint4 *>(vb + voff1);
                const uint4 w2 = *reinterpret_cast<const uint4 *>(vb + voff0 + 8 * kHeadDim);
                const uint4 w3 = *reinterpret_cast<const uint4 *>(vb + voff1 + 8 * kHeadDim);
                const uint32_t a0[4] = {w0.x, w0.y, w0.z, w0.w}, a1[4] = {w1.x, w1.y, w1.z, w1.w};
                const uint32_t a2[4] = {w2.x, w2.y, w2.z, w2.w}, a3[4] = {w3.x, w3.y, w3.z, w3.w};
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const uint32_t x01 = __byte_perm(a0[q4], a1[q4], 0x5410), x23 = __byte_perm(a0[q4], a1[q4], 0x7632);
                    const uint32_t y01 = __byte_perm(a2[q4], a3[q4], 0x5410), y23 = __byte_perm(a2[q4], a3[q4], 0x7632);
                    mma_f16_16816(o[4 * q4 + 0], pa[ks], cvt_bytes02(x01), cvt_bytes02(y01));
                    mma_f16_16816(o[4 * q4 + 1], pa[ks], cvt_bytes13(x01), cvt_bytes13(y01));
                    mma_f16_16816(o[4 * q4 + 2], pa[ks], cvt_bytes02(x23), cvt_bytes02(y23));
                    mma_f16_16816(o[4 * q4 + 3], pa[ks], cvt_bytes13(x23), cvt_bytes13(y23));
                }
            }
        }
    }

    // ---- this warp's partial (m, l, O) into its own buffer; O row r, dim d at r*144 + (d/32)*36 + d%32
    __syncwarp();
    float *ow = reinterpret_cast<float *>(wb.k);   // spans k and v: 16 KB >= 16 * 144 * 4
    float *mw = wb.ks, *lw = wb.vs;
#pragma unroll
    for (int r = 0; r < (ROWS > 8 ? 2 : 1); ++r) {
        const int row = g + 8 * r;
        if (row < p.G) {
            float *dst = ow + row * kORowStride + t * 36;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                *reinterpret_cast<float4 *>(dst + 4 * i) =
                    make_float4(o[4 * i][2 * r], o[4 * i + 1][2 * r], o[4 * i + 2][2 * r], o[4 * i + 3][2 * r]);
                *reinterpret_cast<float4 *>(dst + 16 + 4 * i) =
                    make_float4(o[4 * i][2 * r + 1], o[4 * i + 1][2 * r + 1], o[4 * i + 2][2 * r + 1], o[4 * i + 3][2 * r + 1]);
            }
            if (t == 0) {
                mw[row] = m_row[r];
                lw[row] = l_row[r];
            }
        }
    }
    __syncthreads();

    // ---- merge the four slices (log-sum-exp identity); thread d writes head dim d of every row
    const WarpBuf *all = reinterpret_cast<const WarpBuf *>(smem);
    const int dpos = (tid >> 5) * 36 + (tid & 31);
    for (int row = 0; row < p.G; ++row) {
        float mm[kDecodeWarps], M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            mm[w] = all[w].ks[row];
            M = fmaxf(M, mm[w]);
        }
        float acc = 0.f, l = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            const float f = fast_exp2(mm[w] - M);   // 0 for an empty slice (m = -inf)
            l = fmaf(all[w].vs[row], f, l);
            acc = fmaf(reinterpret_cast<const float *>(all[w].k)[row * kORowStride + dpos], f, acc);
        }
        const size_t slot = ((size_t)b * p.Hq + h0 + row) * p.n_chunks + chunk;
        p.part_o[slot * kHeadDim + tid] = acc;
        if (tid == 0) {
            p.part_ml[slot * 2] = M;
            p.part_ml[slot * 2 + 1] = l;
        }
    }
}

// Second pass: log-sum-exp merge of a row's chunk partials,
//   M = max m_c;  l = sum l_c 2^(m_c - M);  o = sum O_c 2^(m_c - M) / l.
// One warp per (sequence, query head); a lane owns four head dims.
__global__ void __launch_bounds__(128)
slim_decode_merge_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                         const int32_t *__restrict__ kv_len, __nv_bfloat16 *__restrict__ out,
                         int B, int Hq, int n_chunks, int chunk_tokens)
{
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5);   // b * Hq + h
    const int lane = threadIdx.x & 31;
    if (row >= B * Hq) return;
    const int b = row / Hq;
    const int len = kv_len[b];
    const int nc = min(n_chunks, (len + chunk_tokens - 1) / chunk_tokens);
    const float *ml = part_ml + (size_t)row * n_chunks * 2;
    const float *po = part_o + (size_t)row * n_chunks * kHeadDim;
    float M = -INFINITY;
    for (int c = lane; c < nc; c += 32) M = fmaxf(M, ml[2 * c]);
    M = warp_max(M);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    for (int c = 0; c < nc; ++c) {
        const float w = exp2f(ml[2 * c] - M);
        l += ml[2 * c + 1] * w;
        const float4 v = *reinterpret_cast<const float4 *>(po + (size_t)c * kHeadDim + 4 * lane);
        acc.x += v.x * w;
        acc.y += v.y * w;
        acc.z += v.z * w;
        acc.w += v.w * w;
    }
    const float inv = (nc > 0) ? 1.f / l : 0.f;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t *>(&lo);
    pk.y = *reinterpret_cast<uint32_t *>(&hi);
    reinterpret_cast<uint2 *>(out + (size_t)row * kHeadDim)[lane] = pk;
}

// ---------------------------------------------------------------- host side
size_t decode_workspace_bytes(int B, int Hq, int Hkv, int max_kv)
{
    (void)Hkv;
    const size_t nc = (size_t)(max_kv + kChunkTok - 1) / kChunkTok;
    return (size_t)B * Hq * nc * (kHeadDim + 2) * sizeof(float);
}

template <int ROWS>
static int launch_split(const DecodeParams &p, int B, cudaStream_t stream)
{
    constexpr int kBytes = kDecodeWarps * (int)sizeof(WarpBuf);
    SLIM_CUDA_TRY(cudaFuncSetAttribute(slim_decode_split_kernel<ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kBytes));
    dim3 grid((unsigned)p.n_chunks, (unsigned)p.Hkv, (unsigned)B);
    slim_decode_split_kernel<ROWS><<<grid, kDecodeThreads, kBytes, stream>>>(p);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
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
    p.scale_log2e = sm_scale * kLog2e;
    p.part_o = static_cast<float *>(workspace);
    p.part_ml = p.part_o + (size_t)B * Hq * p.n_chunks * kHeadDim;
    return p;
}

int launch_decode_split(const slim_cache_t *c, const void *q, const int32_t *kv_len, int B, int max_kv, int Hq,
                        float sm_scale, void *workspace, cudaStream_t stream)
{
    int C;
    const DecodeParams p = make_params(c, q, kv_len, B, max_kv, Hq, sm_scale, workspace, C);
    if (p.n_chunks == 0) return SLIM_OK;
    return p.G <= 8 ? launch_split<8>(p, B, stream) : launch_split<16>(p, B, stream);
}

int launch_decode_merge(const slim_cache_t *c, void *out, const int32_t *kv_len, int B, int max_kv, int Hq,
                        const void *workspace, cudaStream_t stream)
{
    int C;
    const DecodeParams p = make_params(c, nullptr, kv_len, B, max_kv, Hq, 1.f, const_cast<void *>(workspace), C);
    const int rows = B * Hq;
    slim_decode_merge_kernel<<<(rows + 3) / 4, 128, 0, stream>>>(p.part_o, p.part_ml, kv_len,
                                                                 static_cast<__nv_bfloat16 *>(out), B, Hq,
                                                                 p.n_chunks, C);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

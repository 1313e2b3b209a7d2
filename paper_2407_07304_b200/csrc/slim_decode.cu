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

template <int ROWS, int CP>
struct DecodeSmem {
    static constexpr int C = CP * kPageTokens;          // tokens per chunk
    static constexpr int PSTRIDE = C + 8;               // halfs; +16 bytes keeps A-fragment reads conflict-free
    static constexpr size_t kOffK = 0;
    static constexpr size_t kOffV = kOffK + (size_t)C * kHeadDim;
    static constexpr size_t kOffKs = kOffV + (size_t)C * kHeadDim;
    static constexpr size_t kOffVs = kOffKs + (size_t)C * 4;
    static constexpr size_t kOffS = kOffVs + (size_t)C * 4;
    static constexpr size_t kOffP = kOffS + (size_t)ROWS * C * 4;
    static constexpr size_t kBytes = kOffP + (size_t)ROWS * PSTRIDE * 2;
};

// ROWS: query heads per kv head, rounded up to 1, 8 or 16.  CP: pages per chunk (1 or 2).
template <int ROWS, int CP>
__global__ void __launch_bounds__(kDecodeThreads)
slim_decode_split_kernel(const DecodeParams p)
{
    using L = DecodeSmem<ROWS, CP>;
    constexpr int C = L::C;
    extern __shared__ __align__(128) unsigned char smem[];
    int8_t *kbuf = reinterpret_cast<int8_t *>(smem + L::kOffK);
    int8_t *vbuf = reinterpret_cast<int8_t *>(smem + L::kOffV);
    float *ksc = reinterpret_cast<float *>(smem + L::kOffKs);
    float *vsc = reinterpret_cast<float *>(smem + L::kOffVs);
    float *S = reinterpret_cast<float *>(smem + L::kOffS);
    __half *P = reinterpret_cast<__half *>(smem + L::kOffP);

    const int chunk = blockIdx.x, head = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int len = min(p.kv_len[b], p.max_pages_per_seq * kPageTokens);
    const int n_tok = min(C, len - chunk * C);   // valid tokens of this chunk
    if (n_tok <= 0) return;

    // ---- ask for the whole chunk: K pages (each with its page's K and V scales), then V pages
    const int32_t *bt = p.block_table + (size_t)b * p.max_pages_per_seq + chunk * CP;
    int page[CP];
#pragma unroll
    for (int pg = 0; pg < CP; ++pg) {
        int id = (pg * kPageTokens < n_tok) ? bt[pg] : 0;
        page[pg] = (id >= 0 && id < p.num_pages) ? id : 0;
    }
#pragma unroll
    for (int kv = 0; kv < 2; ++kv) {
#pragma unroll
        for (int pg = 0; pg < CP; ++pg) {
            const int rows = max(0, min(kPageTokens, n_tok - pg * kPageTokens));
            const int8_t *src = p.codes + code_block_offset(page[pg], head, kv, p.Hkv);
            const uint32_t dst = smem_u32((kv ? vbuf : kbuf) + pg * kPageTokens * kHeadDim);
            for (int i = tid; i < rows * 8; i += kDecodeThreads) {
                const int r = i >> 3, c = i & 7;
                cp_async16(dst + swz_row_piece(r, c), src + r * kHeadDim + c * 16);
            }
            if (kv == 0) {
                const int quads = (rows + 3) >> 2;
                for (int i = tid; i < 2 * quads; i += kDecodeThreads) {
                    const int which = i >= quads;
                    const int qd = which ? i - quads : i;
                    const float *ssrc = p.scales + scale_block_offset(page[pg], head, which, p.Hkv) + qd * 4;
                    cp_async16(smem_u32((which ? vsc : ksc) + pg * kPageTokens + qd * 4), ssrc);
                }
            }
            cp_async_commit();
        }
    }

    // ---- query fragments (rows = the G heads of this kv head), while the copies fly
    const int h0 = head * p.G;
    const __nv_bfloat16 *qbase = p.q + ((size_t)b * p.Hq + h0) * kHeadDim;
    QFrag qf;
    float pow2_lo, pow2_hi;
    load_q_frag(qf, (g < p.G) ? qbase + (size_t)g * kHeadDim : nullptr,
                (ROWS > 8 && g + 8 < p.G) ? qbase + (size_t)(g + 8) * kHeadDim : nullptr, t, pow2_lo, pow2_hi);
    const float rs_lo = pow2_lo * p.scale_log2e, rs_hi = pow2_hi * p.scale_log2e;

    // ---- scores of the whole chunk -> S (log2 units)
    auto score_page = [&](int pg) {
        const int rows = n_tok - pg * kPageTokens;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int tok0 = pg * kPageTokens + (warp * 4 + i) * 8;
            if (tok0 - pg * kPageTokens >= rows) break;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            qk_tile(acc, qf, kbuf, tok0, g, t);
            const float2 sk = *reinterpret_cast<const float2 *>(ksc + tok0 + 2 * t);
            const float2 sv = *reinterpret_cast<const float2 *>(vsc + tok0 + 2 * t);
            const float lx = log2_scale(sv.x), ly = log2_scale(sv.y);
            if (ROWS == 1) {
                if (g == 0)
                    *reinterpret_cast<float2 *>(S + tok0 + 2 * t) =
                        make_float2(fmaf(acc[0], sk.x * rs_lo, lx), fmaf(acc[1], sk.y * rs_lo, ly));
            } else {
                *reinterpret_cast<float2 *>(S + g * C + tok0 + 2 * t) =
                    make_float2(fmaf(acc[0], sk.x * rs_lo, lx), fmaf(acc[1], sk.y * rs_lo, ly));
                if (ROWS > 8)
                    *reinterpret_cast<float2 *>(S + (g + 8) * C + tok0 + 2 * t) =
                        make_float2(fmaf(acc[2], sk.x * rs_hi, lx), fmaf(acc[3], sk.y * rs_hi, ly));
            }
        }
    };
    if (CP == 1) {
        cp_async_wait<1>();
        __syncthreads();
        score_page(0);
    } else {
        cp_async_wait<3>();
        __syncthreads();
        score_page(0);
        cp_async_wait<2>();
        __syncthreads();
        if (n_tok > kPageTokens) score_page(1);
    }
    __syncthreads();

    // ---- one softmax per row over the chunk: P = 2^(s' - m') in fp16, l = sum P / scale_v in fp32
    const int n_pad = (n_tok + 15) & ~15;
    for (int r = warp; r < ROWS; r += 4) {
        if (r >= p.G) break;
        float m = -INFINITY;
        for (int i = lane; i < n_tok; i += 32) m = fmaxf(m, S[r * C + i]);
        m = warp_max(m);
        float l = 0.f;
        for (int i = lane; i < n_pad; i += 32) {
            float e = 0.f;
            if (i < n_tok) {
                e = exp2f(S[r * C + i] - m);
                l = fmaf(e, recip_scale(vsc[i]), l);
            }
            P[r * L::PSTRIDE + i] = __float2half_rn(e);
        }
        l = warp_sum(l);
        if (lane == 0) {
            float *ml = p.part_ml + (((size_t)b * p.Hq + h0 + r) * p.n_chunks + chunk) * 2;
            ml[0] = m;
            ml[1] = l;
        }
    }

    // ---- O = P . V: warp w owns head dims [32w, 32w+32); contraction over tokens in steps of 16
    float o[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
    const int piece = 2 * warp + (g >> 2);
    const int inner = (g & 3) * 4;
    auto pv_page = [&](int pg) {
        const int rows = n_tok - pg * kPageTokens;
#pragma unroll 2
        for (int ks = 0; ks < 8; ++ks) {
            if (ks * 16 >= rows) break;
            const int tok0 = pg * kPageTokens + ks * 16;
            uint32_t a[4] = {0u, 0u, 0u, 0u};
            if (g < p.G) {
                a[0] = *reinterpret_cast<const uint32_t *>(P + g * L::PSTRIDE + tok0 + 2 * t);
                a[2] = *reinterpret_cast<const uint32_t *>(P + g * L::PSTRIDE + tok0 + 2 * t + 8);
            }
            if (ROWS > 8 && g + 8 < p.G) {
                a[1] = *reinterpret_cast<const uint32_t *>(P + (g + 8) * L::PSTRIDE + tok0 + 2 * t);
                a[3] = *reinterpret_cast<const uint32_t *>(P + (g + 8) * L::PSTRIDE + tok0 + 2 * t + 8);
            }
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = tok0 + 2 * t + (i & 1) + (i >> 1) * 8;
                // rows past the chunk's last token hold stale bytes: any byte converts to a finite
                // fp16 and its P entry is zero, so they add nothing
                w[i] = *reinterpret_cast<const uint32_t *>(vbuf + swz_row_piece(row, piece) + inner);
            }
            const uint32_t x01 = __byte_perm(w[0], w[1], 0x5410), x23 = __byte_perm(w[0], w[1], 0x7632);
            const uint32_t y01 = __byte_perm(w[2], w[3], 0x5410), y23 = __byte_perm(w[2], w[3], 0x7632);
            mma_f16_16816(o[0], a, cvt_bytes02(x01), cvt_bytes02(y01));
            mma_f16_16816(o[1], a, cvt_bytes13(x01), cvt_bytes13(y01));
            mma_f16_16816(o[2], a, cvt_bytes02(x23), cvt_bytes02(y23));
            mma_f16_16816(o[3], a, cvt_bytes13(x23), cvt_bytes13(y23));
        }
    };
    if (CP == 1) {
        cp_async_wait<0>();
        __syncthreads();
        pv_page(0);
    } else {
        cp_async_wait<1>();
        __syncthreads();
        pv_page(0);
        cp_async_wait<0>();
        __syncthreads();
        if (n_tok > kPageTokens) pv_page(1);
    }

    // ---- unnormalised partial output; thread (g, t) holds dims 32w + 8t + [0, 8) of rows g and g + 8
    const int d0 = 32 * warp + 8 * t;
    if (g < p.G) {
        float *dst = p.part_o + (((size_t)b * p.Hq + h0 + g) * p.n_chunks + chunk) * kHeadDim + d0;
        *reinterpret_cast<float4 *>(dst) = make_float4(o[0][0], o[1][0], o[2][0], o[3][0]);
        *reinterpret_cast<float4 *>(dst + 4) = make_float4(o[0][1], o[1][1], o[2][1], o[3][1]);
    }
    if (ROWS > 8 && g + 8 < p.G) {
        float *dst = p.part_o + (((size_t)b * p.Hq + h0 + g + 8) * p.n_chunks + chunk) * kHeadDim + d0;
        *reinterpret_cast<float4 *>(dst) = make_float4(o[0][2], o[1][2], o[2][2], o[3][2]);
        *reinterpret_cast<float4 *>(dst + 4) = make_float4(o[0][3], o[1][3], o[2][3], o[3][3]);
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
int decode_chunk_pages(int B, int Hkv, int max_kv)
{
    // Two pages per chunk halves the partial traffic; one page per chunk gives short
    // problems enough blocks to fill 148 SMs several times over.
    const long long blocks2 = (long long)B * Hkv * ((max_kv + 255) / 256);
    return blocks2 >= 4LL * 148 ? 2 : 1;
}

size_t decode_workspace_bytes(int B, int Hq, int Hkv, int max_kv)
{
    const int cp = decode_chunk_pages(B, Hkv, max_kv);
    const size_t nc = (size_t)(max_kv + cp * kPageTokens - 1) / (cp * kPageTokens);
    return (size_t)B * Hq * nc * (kHeadDim + 2) * sizeof(float);
}

template <int ROWS, int CP>
static int launch_split(const DecodeParams &p, int B, cudaStream_t stream)
{
    using L = DecodeSmem<ROWS, CP>;
    SLIM_CUDA_TRY(cudaFuncSetAttribute(slim_decode_split_kernel<ROWS, CP>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::kBytes));
    dim3 grid((unsigned)p.n_chunks, (unsigned)p.Hkv, (unsigned)B);
    slim_decode_split_kernel<ROWS, CP><<<grid, kDecodeThreads, L::kBytes, stream>>>(p);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

static DecodeParams make_params(const slim_cache_t *c, const void *q, const int32_t *kv_len, int B, int max_kv,
                                int Hq, float sm_scale, void *workspace, int &C)
{
    const int Hkv = c->num_kv_heads;
    const int cp = decode_chunk_pages(B, Hkv, max_kv);
    C = cp * kPageTokens;
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
    const int cp = C / kPageTokens;
    if (p.G == 1) return cp == 2 ? launch_split<1, 2>(p, B, stream) : launch_split<1, 1>(p, B, stream);
    if (p.G <= 8) return cp == 2 ? launch_split<8, 2>(p, B, stream) : launch_split<8, 1>(p, B, stream);
    return cp == 2 ? launch_split<16, 2>(p, B, stream) : launch_split<16, 1>(p, B, stream);
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

// Causal prefill attention over the INT8 KV cache, warp-level MMA version.
//
// A thread block owns 64 query rows of one query head (16 per warp) and every key
// they can see (the one-dimensional decomposition of Section 2.1: no key split,
// no cross-block merge).  A 64-row score strip over all keys does not fit on
// chip at long sequence lengths, so key tiles of 64 tokens stream through one
// score buffer (registers) with a running row maximum; the result is the same
// softmax attention.  INT8 tiles arrive by 16-byte asynchronous copies, are
// converted to fp16 in registers (Section 2.2 hybrid-dtype step) and feed
// mma.sync tensor-core tiles.
//
// The V scale of key j is folded into the softmax weight: with
//   s'_j = s_j + log2(scale_v[j]),  m' = running max of s',  P_j = 2^(s'_j - m')
// the output is  o = (sum_j P_j * v_code_j) / (sum_j P_j / scale_v[j]),
// identical to softmax(s) . (v_code * scale_v) because the factor 2^(-m') cancels.
#include "slim_common.cuh"

namespace slim {

constexpr int kPfThreads = 128;
constexpr int kPfBM = 64;   // query rows per block
constexpr int kPfBN = 64;   // keys per tile

struct PrefillParams {
    const int8_t *codes;
    const float *scales;
    const int32_t *block_table;
    const int32_t *cu_q;
    const int32_t *kv_len;
    const __nv_bfloat16 *q;   // [total_q][Hq][128]
    __nv_bfloat16 *out;       // [total_q][Hq][128]
    int Hq, Hkv, G, max_pages_per_seq, num_pages, n_qtiles;
    float scale_log2e;
};

struct PfStage {
    int8_t k[kPfBN * kHeadDim];
    int8_t v[kPfBN * kHeadDim];
    float ks[kPfBN];
    float vs[kPfBN];
};

__global__ void __launch_bounds__(kPfThreads)
slim_prefill_mma_kernel(const PrefillParams p)
{
    __shared__ __align__(128) PfStage stage[2];
    const int qtile = p.n_qtiles - 1 - blockIdx.x;   // longest rows first
    const int h = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int q0 = p.cu_q[b];
    const int q_len = p.cu_q[b + 1] - q0;
    const int m0 = qtile * kPfBM;
    if (m0 >= q_len) return;
    const int kvl = min(p.kv_len[b], p.max_pages_per_seq * kPageTokens);
    const int offset = kvl - q_len;                                  // row r sees keys j <= offset + r
    const int n_keys = min(kvl, offset + min(m0 + kPfBM, q_len));    // keys visible to the tile's last row
    const int n_tiles = n_keys > 0 ? (n_keys + kPfBN - 1) / kPfBN : 0;
    const int head = h / p.G;
    const int32_t *bt = p.block_table + (size_t)b * p.max_pages_per_seq;

    auto issue = [&](int kt) {
        PfStage &st = stage[kt & 1];
        const int tok0 = kt * kPfBN;
        const int rows = min(kPfBN, n_keys - tok0);
        int page = bt[tok0 >> 7];
        page = (page >= 0 && page < p.num_pages) ? page : 0;
        const int slot0 = tok0 & (kPageTokens - 1);
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
            const int8_t *src = p.codes + code_block_offset(page, head, kv, p.Hkv) + (size_t)slot0 * kHeadDim;
            const uint32_t dst = smem_u32(kv ? st.v : st.k);
            for (int i = tid; i < rows * 8; i += kPfThreads) {
                const int r = i >> 3, c = i & 7;
                cp_async16(dst + swz_row_piece(r, c), src + r * kHeadDim + c * 16);
            }
            const float *ssrc = p.scales + scale_block_offset(page, head, kv, p.Hkv) + slot0;
            if (tid < ((rows + 3) >> 2)) cp_async16(smem_u32((kv ? st.vs : st.ks) + tid * 4), ssrc + tid * 4);
        }
        cp_async_commit();
    };

    if (n_tiles > 0) issue(0);

    // query fragments of this warp's 16 rows
    const int r_lo = m0 + warp * 16 + g, r_hi = r_lo + 8;
    QFrag qf;
    float pow2_lo, pow2_hi;
    load_q_frag(qf, r_lo < q_len ? p.q + ((size_t)(q0 + r_lo) * p.Hq + h) * kHeadDim : nullptr,
                r_hi < q_len ? p.q + ((size_t)(q0 + r_hi) * p.Hq + h) * kHeadDim : nullptr, t, pow2_lo, pow2_hi);
    const float rs[2] = {pow2_lo * p.scale_log2e, pow2_hi * p.scale_log2e};
    const int last_key[2] = {offset + r_lo, offset + r_hi};   // last visible key of each row

    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) o[i][j] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    for (int kt = 0; kt < n_tiles; ++kt) {
        if (kt + 1 < n_tiles) {
            issue(kt + 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const PfStage &st = stage[kt & 1];
        const int tok0 = kt * kPfBN;
        const int rows = min(kPfBN, n_keys - tok0);

        // ---- scores of this key tile for the warp's 16 rows
        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int j = 0; j < 4; ++j) s[nt][j] = 0.f;
            if (nt * 8 < rows) qk_tile(s[nt], qf, st.k, nt * 8, g, t);
        }
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float2 sk = *reinterpret_cast<const float2 *>(st.ks + nt * 8 + 2 * t);
            const float2 sv = *reinterpret_cast<const float2 *>(st.vs + nt * 8 + 2 * t);
            const float lsv[2] = {log2_scale(sv.x), log2_scale(sv.y)};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int key = tok0 + nt * 8 + 2 * t + (j & 1);
                const int r = j >> 1;
                const float v = fmaf(s[nt][j], ((j & 1) ? sk.y : sk.x) * rs[r], lsv[j & 1]);
                s[nt][j] = (key <= last_key[r] && key < n_keys) ? v : -INFINITY;
                mx[r] = fmaxf(mx[r], s[nt][j]);
            }
        }
        // ---- running maximum and rescale of the accumulators
        float msafe[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float m_new = fmaxf(m_run[r], mx[r]);
            msafe[r] = (m_new == -INFINITY) ? 0.f : m_new;
            const float corr = exp2f(m_run[r] - msafe[r]);
            m_run[r] = m_new;
            l_run[r] *= corr;
#pragma unroll
            for (int nd = 0; nd < 16; ++nd) {
                o[nd][2 * r] *= corr;
                o[nd][2 * r + 1] *= corr;
            }
        }
        // ---- P = 2^(s' - m') to fp16 A-fragments; l += P / scale_v in fp32
        uint32_t pa[4][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float2 sv = *reinterpret_cast<const float2 *>(st.vs + nt * 8 + 2 * t);
            float pv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = j >> 1;
                const bool vis = s[nt][j] != -INFINITY;
                pv[j] = vis ? exp2f(s[nt][j] - msafe[r]) : 0.f;
                if (vis) l_run[r] = fmaf(pv[j], recip_scale((j & 1) ? sv.y : sv.x), l_run[r]);
            }
            pa[nt >> 1][(nt & 1) * 2 + 0] = pack_half2(pv[0], pv[1]);
            pa[nt >> 1][(nt & 1) * 2 + 1] = pack_half2(pv[2], pv[3]);
        }
        // ---- O += P . V ; thread (g, t) supplies head dims 16g + [0, 16) of four token rows per k-step
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            if (ks * 16 < rows) {
                uint4 w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = ks * 16 + 2 * t + (i & 1) + (i >> 1) * 8;
                    w[i] = *reinterpret_cast<const uint4 *>(st.v + swz_row_piece(row, g));
                }
                const uint32_t w0[4] = {w[0].x, w[0].y, w[0].z, w[0].w};
                const uint32_t w1[4] = {w[1].x, w[1].y, w[1].z, w[1].w};
                const uint32_t w2[4] = {w[2].x, w[2].y, w[2].z, w[2].w};
                const uint32_t w3[4] = {w[3].x, w[3].y, w[3].z, w[3].w};
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const uint32_t x01 = __byte_perm(w0[q4], w1[q4], 0x5410), x23 = __byte_perm(w0[q4], w1[q4], 0x7632);
                    const uint32_t y01 = __byte_perm(w2[q4], w3[q4], 0x5410), y23 = __byte_perm(w2[q4], w3[q4], 0x7632);
                    mma_f16_16816(o[4 * q4 + 0], pa[ks], cvt_bytes02(x01), cvt_bytes02(y01));
                    mma_f16_16816(o[4 * q4 + 1], pa[ks], cvt_bytes13(x01), cvt_bytes13(y01));
                    mma_f16_16816(o[4 * q4 + 2], pa[ks], cvt_bytes02(x23), cvt_bytes02(y23));
                    mma_f16_16816(o[4 * q4 + 3], pa[ks], cvt_bytes13(x23), cvt_bytes13(y23));
                }
            }
        }
        __syncthreads();   // everyone is done with this stage before it is refilled
    }

    // ---- normalise and store: thread (g, t) holds dims 32t + [0, 32) of rows r_lo and r_hi
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = r ? r_hi : r_lo;
        float l = l_run[r];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        if (row >= q_len) continue;
        const float f = (l > 0.f) ? 1.f / l : 0.f;
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            __nv_bfloat162 a = __floats2bfloat162_rn(o[2 * i][2 * r] * f, o[2 * i + 1][2 * r] * f);
            __nv_bfloat162 c = __floats2bfloat162_rn(o[2 * i][2 * r + 1] * f, o[2 * i + 1][2 * r + 1] * f);
            pk[i] = *reinterpret_cast<uint32_t *>(&a);
            pk[8 + i] = *reinterpret_cast<uint32_t *>(&c);
        }
        uint4 *dst = reinterpret_cast<uint4 *>(p.out + ((size_t)(q0 + row) * p.Hq + h) * kHeadDim + 32 * t);
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
    }
}

int launch_prefill_mma(const slim_cache_t *c, const void *q, void *out, const int32_t *cu_q, const int32_t *kv_len,
                       int B, int max_q, int Hq, float sm_scale, cudaStream_t stream)
{
    PrefillParams p;
    p.codes = c->codes;
    p.scales = c->scales;
    p.block_table = c->block_table;
    p.cu_q = cu_q;
    p.kv_len = kv_len;
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.Hq = Hq;
    p.Hkv = c->num_kv_heads;
    p.G = Hq / c->num_kv_heads;
    p.max_pages_per_seq = c->max_pages_per_seq;
    p.num_pages = c->num_pages;
    p.n_qtiles = (max_q + kPfBM - 1) / kPfBM;
    p.scale_log2e = sm_scale * kLog2e;
    if (p.n_qtiles == 0) return SLIM_OK;
    dim3 grid((unsigned)p.n_qtiles, (unsigned)Hq, (unsigned)B);
    slim_prefill_mma_kernel<<<grid, kPfThreads, 0, stream>>>(p);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

// Decode split pass on the 5th-generation tensor cores (tcgen05, accumulators in tensor memory).
//
// The next-token phase is bound by memory bandwidth (Section 2.2, Eq. 1: every cached byte is read
// once per generated token), so the kernel is built to spend almost no instructions per cached byte:
//
//  * A thread block owns 256 consecutive tokens (two 128-token tiles) of one (sequence, kv head).  All
//    of its K rows, V rows and scales are requested at once with 16-byte asynchronous copies and land
//    in shared memory in the 128-byte-swizzled layout the tensor cores read directly.
//  * Scores: S^T[token][head] = K_codes[128 x 128] . Q^T by tcgen05.mma kind::i8 - the INT8 codes are the
//    A operand as they are (no dequantisation pass, Section 2.2's hybrid-dtype step happens inside the
//    tensor core).  Q is a 14-bit fixed-point copy split into two signed bytes per value; the G = Hq/Hkv
//    heads of the kv head give 2G (padded to 16 or 32) MMA columns: [high bytes | low bytes].
//  * One softmax over the block's 256 scores per head (Section 2.1 order: all scores, softmax, then .V),
//    with thread = token after a tensor-memory load.
//  * Output: O^T[dim][head] = V_codes^T[128 x 256] . P^T, again kind::i8, the V tile read MN-major
//    straight from its token-major rows; P is 16-bit fixed point split into two unsigned bytes.
//  * 256 * high + low is recombined exactly in int32; one partial (m, l, O[128]) per (head, block).
//
// The V scale is folded into the softmax weight (s'_j = s_j + log2 sv_j, P_j = 2^(s'_j - max s'),
// o = sum P_j c_j / sum P_j / sv_j), so P <= 1 is normalised by the block's largest contribution.
#include "slim_common.cuh"
#include "slim_decode_params.cuh"
#include "slim_tcgen05.cuh"

namespace slim {

constexpr int kTcThreads = 128;
constexpr int kTileTok = 128;
constexpr int kTcChunkTok = 2 * kTileTok;
constexpr float kQFixTc = 8192.f;      // |q / pow2| < 2  ->  |v| < 16384, high byte in [-64, 64]
constexpr float kPFixTc = 65535.f;
constexpr uint32_t kTmemCols = 128;

template <int NH>
struct TcSmem {
    static constexpr int N = 2 * NH;                       // MMA columns: [hi bytes of NH heads | lo bytes]
    static constexpr uint32_t kOffK = 0;                   // two K tiles, 16 KB each (1024-byte aligned)
    static constexpr uint32_t kOffV = 32768;               // two V tiles
    static constexpr uint32_t kOffQ = 65536;               // Q operand: N rows x 128 bytes, core-matrix layout
    static constexpr uint32_t kOffKs = kOffQ + N * 128;    // 256 K scales
    static constexpr uint32_t kOffVs = kOffKs + 1024;      // 256 V scales
    static constexpr uint32_t kOffRed = kOffVs + 1024;     // [4 warps][16] maxima, [4][16] sums, [16] row scales
    static constexpr uint32_t kOffBar = kOffRed + (64 + 64 + 16) * 4;   // two mbarriers, tmem address
    static constexpr uint32_t kBytes = kOffBar + 32;
    static constexpr uint32_t kPTileBytes = N * 128;       // a P^T tile (aliases the K tiles once they are consumed)
};

// Byte offset of element (row n, k byte kb) of a K-major operand stored as 8x16-byte core matrices:
// 16 bytes of k contiguous, 8 rows 16 bytes apart, next 16 k-bytes +128, next 8 rows +1024.
__device__ __forceinline__ uint32_t core_off(int n, int kb)
{
    return (uint32_t)((n >> 3) * 1024 + (kb >> 4) * 128 + (n & 7) * 16 + (kb & 15));
}

template <int NH>
__global__ void __launch_bounds__(kTcThreads)
slim_decode_split_tc_kernel(const DecodeParams p)
{
    using L = TcSmem<NH>;
    constexpr int N = L::N;
    extern __shared__ __align__(1024) unsigned char smem[];
    const int chunk = blockIdx.x, head = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // the page ids do not depend on the length: ask for both at once (two dependent round trips otherwise)
    const int32_t *bt = p.block_table + (size_t)b * p.max_pages_per_seq + chunk * 2;
    const int id0 = (chunk * 2 < p.max_pages_per_seq) ? __ldg(bt) : 0;
    const int id1 = (chunk * 2 + 1 < p.max_pages_per_seq) ? __ldg(bt + 1) : 0;
    const int len = min(__ldg(p.kv_len + b), p.max_pages_per_seq * kPageTokens);
    const int n_tok = min(kTcChunkTok, len - chunk * kTcChunkTok);   // valid tokens of this block
    if (n_tok <= 0) return;
    const int n_tiles = n_tok > kTileTok ? 2 : 1;
    const int h0 = head * p.G;

    float *ks_s = reinterpret_cast<float *>(smem + L::kOffKs);
    float *vs_s = reinterpret_cast<float *>(smem + L::kOffVs);
    float *red_m = reinterpret_cast<float *>(smem + L::kOffRed);
    float *red_l = red_m + 64;
    float *rowscale = red_l + 64;
    const uint32_t bar_qk = smem_u32(smem + L::kOffBar), bar_pv = bar_qk + 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kOffBar + 16);
    const uint32_t smem_base = smem_u32(smem);

    // ---- ask for the whole block: K tile 0 + its scales | K tile 1 + scales | V tile 0 | V tile 1
    {
        int page[2] = {id0, id1};
#pragma unroll
        for (int t = 0; t < 2; ++t) page[t] = (page[t] >= 0 && page[t] < p.num_pages) ? page[t] : 0;
        const int r0 = tid >> 3, c = tid & 7;
        const uint32_t dsw = (uint32_t)(r0 * kHeadDim + ((c ^ (r0 & 7)) << 4));   // rows r0 + 16 * it keep (row & 7)
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int rows = min(kTileTok, n_tok - t * kTileTok);
                const int8_t *src = p.codes + code_block_offset(page[t], head, kv, p.Hkv) + r0 * kHeadDim + c * 16;
                const uint32_t dst = smem_base + (kv ? L::kOffV : L::kOffK) + t * 16384 + dsw;
#pragma unroll
                for (int it = 0; it < 8; ++it)
                    if (r0 + 16 * it < rows) cp_async16(dst + it * 16 * kHeadDim, src + it * 16 * kHeadDim);
                if (kv == 0 && tid < 64) {
                    const int which = tid >> 5, qd = tid & 31;
                    if (qd * 4 < rows)
                        cp_async16(smem_u32((which ? vs_s : ks_s) + t * kTileTok + qd * 4),
                                   p.scales + scale_block_offset(page[t], head, which, p.Hkv) + qd * 4);
                }
                cp_async_commit();
            }
        }
    }

    // ---- set-up while the copies fly: barriers, tensor memory, the fixed-point Q operand
    if (tid == 0) {
        tc::mbar_init(bar_qk, 1);
        tc::mbar_init(bar_pv, 1);
        tc::mbar_init_fence();
    }
    if (warp == 0) tc::tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    {
        // warp w converts heads w, w+4, ...; a lane owns four consecutive dims.  Rows of unused heads are zero.
        const __nv_bfloat16 *qbase = p.q + ((size_t)b * p.Hq + h0) * kHeadDim;
        for (int h = warp; h < NH; h += 4) {
            uint32_t lo_w = 0, hi_w = 0;
            if (h < p.G) {
                const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(qbase + (size_t)h * kHeadDim) + lane);
                float x[4] = {bf16_bits_to_float(raw.x & 0xFFFFu), bf16_bits_to_float(raw.x >> 16),
                              bf16_bits_to_float(raw.y & 0xFFFFu), bf16_bits_to_float(raw.y >> 16)};
                const float am = warp_max(fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3]))));
                const float p2 = pow2_floor(am);
                const float f = pow2_recip(p2) * kQFixTc;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    // v = round(x * f), |v| < 16384, as the low 16 bits of 1.5 * 2^23 + v (two's complement)
                    const int v = (int)(int16_t)(__float_as_uint(fmaf(x[i], f, 12582912.f)) & 0xFFFFu);
                    const int hi = (v + 128) >> 8;            // v = 256 * hi + lo with lo in [-128, 127]
                    lo_w |= ((uint32_t)v & 0xFFu) << (8 * i);
                    hi_w |= ((uint32_t)hi & 0xFFu) << (8 * i);
                }
                if (lane == 0) rowscale[h] = p2 * p.scale_log2e * (1.f / kQFixTc);
            }
            *reinterpret_cast<uint32_t *>(smem + L::kOffQ + core_off(h, 4 * lane)) = hi_w;
            *reinterpret_cast<uint32_t *>(smem + L::kOffQ + core_off(NH + h, 4 * lane)) = lo_w;
        }
    }

    // ---- K tiles and scales have landed: scores on the tensor cores
    cp_async_wait<2>();
    tc::fence_proxy_async();
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;
    if (tid == 0) {
        constexpr uint32_t idesc = tc::instr_desc(2, 1, 1, false, false, 128, N);   // s32 <- s8 (K-major) x s8 (K-major)
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            if (t < n_tiles) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint64_t a = tc::smem_desc(smem_base + L::kOffK + t * 16384 + j * 32, 16, 1024, tc::kSwizzle128B);
                    const uint64_t bq = tc::smem_desc(smem_base + L::kOffQ + j * 256, 128, 1024, tc::kSwizzleNone);
                    tc::mma_i8(tmem + t * N, a, bq, idesc, j > 0);
                }
            }
        }
        tc::commit(bar_qk);
    }

    // this thread's tokens: tid (tile 0) and 128 + tid (tile 1)
    float sk[2], lsv[2], rsv[2];
    bool valid[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int tok = t * kTileTok + tid;
        valid[t] = tok < n_tok;
        const float sv = valid[t] ? fmaxf(vs_s[tok], kMinScale) : 1.f;
        sk[t] = valid[t] ? ks_s[tok] : 0.f;
        lsv[t] = __log2f(sv);
        rsv[t] = valid[t] ? __frcp_rn(sv) : 0.f;
    }

    ok = tc::mbar_wait(bar_qk, 0);
    __syncwarp();   // reconverge after the wait loop: the tensor-memory load below is warp-aligned
    tc::fence_after_sync();

    // ---- S^T from tensor memory: row = token, columns [hi | lo] per head
    float s[2][NH];
    float mloc[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) mloc[h] = -INFINITY;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        if (t < n_tiles) {
            uint32_t r[N];
#pragma unroll
            for (int c16 = 0; c16 < N / 16; ++c16) {
                uint32_t tmp[16];
                tc::tmem_ld16(tmem + lane_base + t * N + c16 * 16, tmp);
#pragma unroll
                for (int i = 0; i < 16; ++i) r[c16 * 16 + i] = tmp[i];
            }
            tc::tmem_ld_wait();
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                const float x = (float)(((int)r[h] << 8) + (int)r[NH + h]);
                s[t][h] = (valid[t] && h < p.G) ? fmaf(x, sk[t] * rowscale[h], lsv[t]) : -INFINITY;
                mloc[h] = fmaxf(mloc[h], s[t][h]);
            }
        } else {
#pragma unroll
            for (int h = 0; h < NH; ++h) s[t][h] = -INFINITY;
        }
    }
#pragma unroll
    for (int h = 0; h < NH; ++h) {
        if (h < p.G) {
            const float m = warp_max(mloc[h]);
            if (lane == 0) red_m[warp * 16 + h] = m;
        }
    }
    tc::fence_before_sync();
    __syncthreads();

    // ---- one softmax over the block's scores per head; P^T (bytes [hi | lo]) into the consumed K tiles
    float lloc[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) {
        lloc[h] = 0.f;
        if (h < p.G) {
            const float M = fmaxf(fmaxf(red_m[h], red_m[16 + h]), fmaxf(red_m[32 + h], red_m[48 + h]));
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (t < n_tiles) {
                    const float e = exp2f(s[t][h] - M);
                    lloc[h] = fmaf(e, rsv[t], lloc[h]);
                    const uint32_t bits = __float_as_uint(fmaf(e, kPFixTc, 8388608.f));   // 2^23 + round(e * 65535)
                    unsigned char *pt = smem + L::kOffK + t * L::kPTileBytes;
                    pt[core_off(h, tid)] = (unsigned char)((bits >> 8) & 0xFFu);
                    pt[core_off(NH + h, tid)] = (unsigned char)(bits & 0xFFu);
                }
            }
            const float l = warp_sum(lloc[h]);
            if (lane == 0) red_l[warp * 16 + h] = l;
        }
    }

    // ---- V tiles have landed: O^T += V^T . P^T on the tensor cores
    cp_async_wait<0>();
    tc::fence_proxy_async();
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    if (tid == 0) {
        constexpr uint32_t idesc = tc::instr_desc(2, 1, 0, true, false, 128, N);   // s32 <- s8 (MN-major) x u8 (K-major)
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            if (t < n_tiles) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint64_t a = tc::smem_desc(smem_base + L::kOffV + t * 16384 + j * 4096, 1024, 1024, tc::kSwizzle128B);
                    const uint64_t bp = tc::smem_desc(smem_base + L::kOffK + t * L::kPTileBytes + j * 256, 128, 1024, tc::kSwizzleNone);
                    tc::mma_i8(tmem + 2 * N, a, bp, idesc, (t > 0) || (j > 0));
                }
            }
        }
        tc::commit(bar_pv);
    }
    ok = tc::mbar_wait(bar_pv, 0) && ok;
    __syncwarp();
    tc::fence_after_sync();

    // ---- O^T from tensor memory: row = head dim, columns [hi | lo] per head; one partial per head
    {
        uint32_t r[N];
#pragma unroll
        for (int c16 = 0; c16 < N / 16; ++c16) {
            uint32_t tmp[16];
            tc::tmem_ld16(tmem + lane_base + 2 * N + c16 * 16, tmp);
#pragma unroll
            for (int i = 0; i < 16; ++i) r[c16 * 16 + i] = tmp[i];
        }
        tc::tmem_ld_wait();
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            if (h < p.G) {
                const size_t slot = ((size_t)b * p.Hq + h0 + h) * p.n_chunks + chunk;
                p.part_o[slot * kHeadDim + tid] = (float)(((int)r[h] << 8) + (int)r[NH + h]) * (1.f / kPFixTc);
            }
        }
    }
    if (tid < p.G) {
        const size_t slot = ((size_t)b * p.Hq + h0 + tid) * p.n_chunks + chunk;
        p.part_ml[slot * 2] = fmaxf(fmaxf(red_m[tid], red_m[16 + tid]), fmaxf(red_m[32 + tid], red_m[48 + tid]));
        p.part_ml[slot * 2 + 1] = red_l[tid] + red_l[16 + tid] + red_l[32 + tid] + red_l[48 + tid];
    }
    if (!ok && p.status != nullptr) atomicExch(p.status, SLIM_ERR_TIMEOUT);
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_dealloc(tmem, kTmemCols);
}

int launch_decode_split_tc(const DecodeParams &p, int B, cudaStream_t stream)
{
    dim3 grid((unsigned)p.n_chunks, (unsigned)p.Hkv, (unsigned)B);
    if (p.G <= 8) {
        constexpr int bytes = (int)TcSmem<8>::kBytes;
        SLIM_CUDA_TRY(cudaFuncSetAttribute(slim_decode_split_tc_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
        slim_decode_split_tc_kernel<8><<<grid, kTcThreads, bytes, stream>>>(p);
    } else {
        constexpr int bytes = (int)TcSmem<16>::kBytes;
        SLIM_CUDA_TRY(cudaFuncSetAttribute(slim_decode_split_tc_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
        slim_decode_split_tc_kernel<16><<<grid, kTcThreads, bytes, stream>>>(p);
    }
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

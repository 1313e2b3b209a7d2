// Decode attention over the INT8 KV cache: split kernel + merge kernel.
//
// The next-token phase is a matrix-vector product bound by memory bandwidth
// (Section 2.2, Eq. 1: every cached byte is read once per generated token), so
// the kernel is organised around keeping the whole key range in flight and
// spending as few instructions per cached byte as possible.
//
//  * A thread block owns 256 consecutive tokens of one (sequence, kv head); each
//    of its four warps owns 64 of them and asks for its K rows, V rows and scales
//    with 16-byte asynchronous copies, all in flight at once.
//  * The INT8 codes go to the tensor cores as they are (integer MMA, m16n8k32):
//    no per-element conversion.  The other operand is a 16-bit fixed-point copy
//    of Q (and later of the softmax weights P) split into a high and a low byte,
//    two integer MMAs per tile, recombined exactly as 256 * hi + lo in int32.
//    The G = Hq / Hkv query heads that share the kv head are the rows of the
//    16-row tile, so each cached byte is used once for all of them.
//  * Inside the block the order is SlimAttention's (Section 2.1): all 256 scores
//    first, one softmax over them, then the product with V - no running rescale.
//
// The V scale of key j is folded into the softmax weight: with
//   s'_j = s_j + log2(scale_v[j]),  m' = max_j s'_j,  P_j = 2^(s'_j - m')
// the output is  o = (sum_j P_j * v_code_j) / (sum_j P_j / scale_v[j]),
// identical to softmax(s) . (v_code * scale_v) because the factor 2^(-m') cancels.
// P_j <= 1 is normalised by the block's largest contribution, which is what
// makes its 16-bit fixed-point copy safe whatever the spread of the V scales.
#include <stdlib.h>

#include "slim_common.cuh"
#include "slim_decode_params.cuh"

namespace slim {

constexpr int kDecodeThreads = 128;
constexpr int kDecodeWarps = 4;
constexpr int kWarpTok = 64;                              // tokens owned by one warp
constexpr int kChunkTok = kDecodeWarps * kWarpTok;        // tokens per thread block (two pages)
constexpr float kQFix = 16384.f;                          // Q fixed point: |q / pow2| < 2  ->  |v| < 32768
constexpr float kPFix = 65535.f;                          // P fixed point: P in [0, 1]     ->  v in [0, 65535]

// Shared memory of one warp: its 64 tokens' K and V rows (swizzled, see swz_row_piece) and
// scales.  After the warp has consumed them the K/V bytes hold its partial result.
struct __align__(128) WarpBuf {
    int8_t k[kWarpTok * kHeadDim];
    int8_t v[kWarpTok * kHeadDim];
    float ks[kWarpTok];
    float vs[kWarpTok];    // V scales, then log2 of them
    float rsv[kWarpTok];   // 1 / V scale
    float red[32];         // [0,16): slice row maxima, [16,32): slice row sums
};
// A warp's partial output lives in its (consumed) K bytes as [row][128] int32 with the 16-byte
// chunk index of dim d XOR-ed by (row ^ 2 * (d / 32)) & 7, which spreads the fragment stores
// over the banks.
__device__ __forceinline__ int opart_word(int row, int d)
{
    return row * kHeadDim + ((((d >> 2) ^ ((row ^ (2 * (d >> 5))) & 7))) << 2) + (d & 3);
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_rcp(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// D(16x8, s32) += A(16x32, s8 or u8, row) * B(32x8, s8, col)
template <bool A_UNSIGNED>
__device__ __forceinline__ void mma_i8_16832(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1)
{
    if (A_UNSIGNED)
        asm volatile(
            "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
            : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Round-to-nearest-even integer of x in [0, 2^22) as the low bits of x + 2^23.
__device__ __forceinline__ uint32_t fix_bits(float x, float scale)
{
    return __float_as_uint(fmaf(x, scale, 8388608.f));
}

// 16-bit fixed-point copy of the query rows as integer-MMA A fragments.
// Thread (g, t) covers head dims [32t, 32t + 32) of rows g and g + 8; MMA step s (0..3)
// contracts dims 32t + 8s + [0, 4) (first half of k) and 32t + 8s + [4, 8) (second half),
// which is the order the K bytes arrive in (two 16-byte pieces per token and thread).
template <bool HI_ROWS>
struct QFix {
    uint32_t hi[HI_ROWS ? 2 : 1][8];   // signed high bytes,   word j = dims 32t + 4j + [0, 4)
    uint32_t lo[HI_ROWS ? 2 : 1][8];   // unsigned low bytes
    float pow2[2];
};

template <bool HI_ROWS>
__device__ __forceinline__ void load_q_fix(QFix<HI_ROWS> &qf, const __nv_bfloat16 *row_lo, const __nv_bfloat16 *row_hi,
                                           int t)
{
    qf.pow2[0] = qf.pow2[1] = 1.f;
#pragma unroll
    for (int r = 0; r < (HI_ROWS ? 2 : 1); ++r) {
        const __nv_bfloat16 *row = r ? row_hi : row_lo;
        float x[32];
        if (row != nullptr) {
            const uint4 *src = reinterpret_cast<const uint4 *>(row + 32 * t);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 v = __ldg(src + i);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    x[i * 8 + 2 * k] = bf16_bits_to_float(w[k] & 0xFFFFu);
                    x[i * 8 + 2 * k + 1] = bf16_bits_to_float(w[k] >> 16);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) x[i] = 0.f;
        }
        float am = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) am = fmaxf(am, fabsf(x[i]));
        am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, 1));
        am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, 2));
        qf.pow2[r] = pow2_floor(am);
        const float f = pow2_recip(qf.pow2[r]) * kQFix;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            // v = round(x * f) in (-32768, 32768): as int16 bits, hi = v >> 8 (signed), lo = v & 255
            uint32_t b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) b[i] = __float_as_uint(fmaf(x[4 * j + i], f, 12582912.f));   // 1.5 * 2^23 + v
            const uint32_t p01 = __byte_perm(b[0], b[1], 0x5140);   // [lo0, lo1, hi0, hi1]
            const uint32_t p23 = __byte_perm(b[2], b[3], 0x5140);
            qf.lo[r][j] = __byte_perm(p01, p23, 0x5410);
            qf.hi[r][j] = __byte_perm(p01, p23, 0x7632);
        }
    }
}

// ROWS: query heads per kv head, rounded up to 8 or 16 (rows of the 16-row MMA tile in use).
template <int ROWS>
__global__ void __launch_bounds__(kDecodeThreads)
slim_decode_split_kernel(const DecodeParams p)
{
    constexpr bool HI = ROWS > 8;
    constexpr int NR = HI ? 2 : 1;
    extern __shared__ __align__(128) unsigned char smem[];
    const int chunk = blockIdx.x, head = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int len = min(p.kv_len[b], p.max_pages_per_seq * kPageTokens);
    const int n_tok = min(kChunkTok, len - chunk * kChunkTok);   // valid tokens of this block
    if (n_tok <= 0) return;
    WarpBuf *all = reinterpret_cast<WarpBuf *>(smem);
    WarpBuf &wb = all[warp];
    const int n_w = max(0, min(kWarpTok, n_tok - warp * kWarpTok));   // valid tokens of this warp
    const int h0 = head * p.G;

    float s[8][2 * NR];           // scores of the slice: s[nt] = tokens 8nt + {2t, 2t+1} of rows g (and g + 8)
    float m_loc[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) m_loc[r] = -INFINITY;

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

        // ---- fixed-point query fragments (rows = the G heads of this kv head), while the copies fly
        const __nv_bfloat16 *qbase = p.q + ((size_t)b * p.Hq + h0) * kHeadDim;
        QFix<HI> qf;
        load_q_fix<HI>(qf, (g < p.G) ? qbase + (size_t)g * kHeadDim : nullptr,
                       (HI && g + 8 < p.G) ? qbase + (size_t)(g + 8) * kHeadDim : nullptr, t);
        float rs[NR];
#pragma unroll
        for (int r = 0; r < NR; ++r) rs[r] = qf.pow2[r] * p.scale_log2e * (1.f / kQFix);

        cp_async_wait<1>();
        __syncwarp();
        // per-token log2 and reciprocal of the V scale, once per token (lane = token)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int tok = lane + 32 * i;
            if (tok < n_w) {
                const float sv = fmaxf(wb.vs[tok], kMinScale);
                wb.vs[tok] = __log2f(sv);
                wb.rsv[tok] = fast_rcp(sv);
            } else {
                wb.rsv[tok] = 0.f;
            }
        }
        __syncwarp();

        // ---- all scores of the slice: integer MMAs straight from the K bytes
        const uint32_t koff0 = (uint32_t)(g * kHeadDim + (((2 * t) ^ g) << 4));
        const uint32_t koff1 = (uint32_t)(g * kHeadDim + (((2 * t + 1) ^ g) << 4));
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            if (nt * 8 < n_w) {
                const int8_t *kb = wb.k + nt * 8 * kHeadDim;
                const uint4 lo4 = *reinterpret_cast<const uint4 *>(kb + koff0);
                const uint4 hi4 = *reinterpret_cast<const uint4 *>(kb + koff1);
                const uint32_t w[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
                int ah[4] = {0, 0, 0, 0}, al[4] = {0, 0, 0, 0};
#pragma unroll
                for (int st = 0; st < 4; ++st) {
                    mma_i8_16832<false>(ah, qf.hi[0][2 * st], HI ? qf.hi[NR - 1][2 * st] : 0u, qf.hi[0][2 * st + 1],
                                        HI ? qf.hi[NR - 1][2 * st + 1] : 0u, w[2 * st], w[2 * st + 1]);
                    mma_i8_16832<true>(al, qf.lo[0][2 * st], HI ? qf.lo[NR - 1][2 * st] : 0u, qf.lo[0][2 * st + 1],
                                       HI ? qf.lo[NR - 1][2 * st + 1] : 0u, w[2 * st], w[2 * st + 1]);
                }
                const float2 sk = *reinterpret_cast<const float2 *>(wb.ks + nt * 8 + 2 * t);
                const float2 lv = *reinterpret_cast<const float2 *>(wb.vs + nt * 8 + 2 * t);
                const bool v0 = nt * 8 + 2 * t < n_w, v1 = nt * 8 + 2 * t + 1 < n_w;
#pragma unroll
                for (int r = 0; r < NR; ++r) {
                    const float x0 = (float)((ah[2 * r] << 8) + al[2 * r]);
                    const float x1 = (float)((ah[2 * r + 1] << 8) + al[2 * r + 1]);
                    s[nt][2 * r] = v0 ? fmaf(x0, sk.x * rs[r], lv.x) : -INFINITY;
                    s[nt][2 * r + 1] = v1 ? fmaf(x1, sk.y * rs[r], lv.y) : -INFINITY;
                    m_loc[r] = fmaxf(m_loc[r], fmaxf(s[nt][2 * r], s[nt][2 * r + 1]));
                }
            } else {
#pragma unroll
                for (int j = 0; j < 2 * NR; ++j) s[nt][j] = -INFINITY;
            }
        }
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            m_loc[r] = fmaxf(m_loc[r], __shfl_xor_sync(0xffffffffu, m_loc[r], 1));
            m_loc[r] = fmaxf(m_loc[r], __shfl_xor_sync(0xffffffffu, m_loc[r], 2));
        }
    }
    // ---- block-wide row maxima
    if (t == 0) {
#pragma unroll
        for (int r = 0; r < NR; ++r) wb.red[g + 8 * r] = m_loc[r];
    }
    __syncthreads();
    float m_blk[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) {
        m_blk[r] = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) m_blk[r] = fmaxf(m_blk[r], all[w].red[g + 8 * r]);
    }

    float l_loc[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) l_loc[r] = 0.f;
    int *ow = reinterpret_cast<int *>(wb.k);   // this warp's partial output: 16 rows x 128 int32 = the K bytes

    if (n_w > 0) {
        // ---- one softmax over the block's 256 scores: P = 2^(s' - m') in 16-bit fixed point, as
        //      high-byte and low-byte A fragments of the two 32-token MMA steps; l = sum P / scale_v
        uint32_t pa_hi[2][2 * NR], pa_lo[2][2 * NR];
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
            for (int r = 0; r < NR; ++r) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    // k slots 4t + {0,1,2,3} <- tokens of tiles (4ks + 2half, 4ks + 2half + 1), columns 2t, 2t+1
                    uint32_t bits[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int nt = 4 * ks + 2 * half + (i >> 1);
                        const float e = fast_exp2(s[nt][2 * r + (i & 1)] - m_blk[r]);
                        l_loc[r] = fmaf(e, wb.rsv[nt * 8 + 2 * t + (i & 1)], l_loc[r]);
                        bits[i] = fix_bits(e, kPFix);
                    }
                    const uint32_t p01 = __byte_perm(bits[0], bits[1], 0x5140);   // [lo0, lo1, hi0, hi1]
                    const uint32_t p23 = __byte_perm(bits[2], bits[3], 0x5140);
                    pa_lo[ks][NR * half + r] = __byte_perm(p01, p23, 0x5410);
                    pa_hi[ks][NR * half + r] = __byte_perm(p01, p23, 0x7632);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            l_loc[r] += __shfl_xor_sync(0xffffffffu, l_loc[r], 1);
            l_loc[r] += __shfl_xor_sync(0xffffffffu, l_loc[r], 2);
        }

        // ---- O = P . V: integer MMAs over 32-token steps.  Thread (g, t) supplies head dims
        //      16g + [0, 16) (one 16-byte piece per token row) of token rows
        //      32ks + {2t, 2t+1, 8+2t, 9+2t} (first half of k) and + 16 (second half); the bytes of
        //      four rows are transposed in registers into per-dim words.  Two passes of eight dims.
        cp_async_wait<0>();
        __syncwarp();
        const uint32_t voff0 = (uint32_t)((2 * t) * kHeadDim + ((g ^ (2 * t)) << 4));
        const uint32_t voff1 = (uint32_t)((2 * t + 1) * kHeadDim + ((g ^ (2 * t + 1)) << 4));
        __syncwarp();
#pragma unroll
        for (int dh = 0; dh < 2; ++dh) {
            int oh[8][4], ol[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) oh[i][j] = ol[i][j] = 0;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                if (ks * 32 < n_w) {
                    // rows past the slice's last token hold stale bytes; their P entries are zero
                    const int8_t *vb = wb.v + ks * 32 * kHeadDim + dh * 8;
                    uint2 rw[8];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        rw[2 * q] = *reinterpret_cast<const uint2 *>(vb + voff0 + q * 8 * kHeadDim);
                        rw[2 * q + 1] = *reinterpret_cast<const uint2 *>(vb + voff1 + q * 8 * kHeadDim);
                    }
#pragma unroll
                    for (int wd = 0; wd < 2; ++wd) {
                        uint32_t bfrag[2][4];   // [k half][dim within the word]
#pragma unroll
                        for (int kh = 0; kh < 2; ++kh) {
                            const uint32_t r0 = wd ? rw[4 * kh].y : rw[4 * kh].x, r1 = wd ? rw[4 * kh + 1].y : rw[4 * kh + 1].x;
                            const uint32_t r2 = wd ? rw[4 * kh + 2].y : rw[4 * kh + 2].x, r3 = wd ? rw[4 * kh + 3].y : rw[4 * kh + 3].x;
                            const uint32_t t0 = __byte_perm(r0, r1, 0x5140), t1 = __byte_perm(r2, r3, 0x5140);
                            const uint32_t t2 = __byte_perm(r0, r1, 0x7362), t3 = __byte_perm(r2, r3, 0x7362);
                            bfrag[kh][0] = __byte_perm(t0, t1, 0x5410);
                            bfrag[kh][1] = __byte_perm(t0, t1, 0x7632);
                            bfrag[kh][2] = __byte_perm(t2, t3, 0x5410);
                            bfrag[kh][3] = __byte_perm(t2, t3, 0x7632);
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            mma_i8_16832<true>(oh[4 * wd + i], pa_hi[ks][0], HI ? pa_hi[ks][NR - 1] : 0u, pa_hi[ks][NR],
                                               HI ? pa_hi[ks][2 * NR - 1] : 0u, bfrag[0][i], bfrag[1][i]);
                            mma_i8_16832<true>(ol[4 * wd + i], pa_lo[ks][0], HI ? pa_lo[ks][NR - 1] : 0u, pa_lo[ks][NR],
                                               HI ? pa_lo[ks][2 * NR - 1] : 0u, bfrag[0][i], bfrag[1][i]);
                        }
                    }
                }
            }
            // this pass's eight dims per column: dims 32t + 16c + 8dh + i for columns n = 2t + c
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                const int row = g + 8 * r;
                if (row < p.G) {
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        int v[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[i] = (oh[i][2 * r + c] << 8) + ol[i][2 * r + c];
                        const int d = 32 * t + 16 * c + 8 * dh;
                        *reinterpret_cast<int4 *>(ow + opart_word(row, d)) = make_int4(v[0], v[1], v[2], v[3]);
                        *reinterpret_cast<int4 *>(ow + opart_word(row, d + 4)) = make_int4(v[4], v[5], v[6], v[7]);
                    }
                }
            }
        }
    } else {
        // an empty slice contributes zeros
        for (int i = lane; i < ROWS * kHeadDim; i += 32) ow[i] = 0;
    }
    if (t == 0) {
#pragma unroll
        for (int r = 0; r < NR; ++r) wb.red[16 + g + 8 * r] = l_loc[r];
    }
    __syncthreads();

    // ---- sum the four slices (same maximum, so integer partial outputs add exactly);
    //      thread d writes head dim d of every row
    for (int row = 0; row < p.G; ++row) {
        const int dpos = opart_word(row, tid) - row * kHeadDim;
        int acc = 0;
        float l = 0.f, M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            acc += reinterpret_cast<const int *>(all[w].k)[row * kHeadDim + dpos];
            l += all[w].red[16 + row];
            M = fmaxf(M, all[w].red[row]);
        }
        const size_t slot = ((size_t)b * p.Hq + h0 + row) * p.n_chunks + chunk;
        p.part_o[slot * kHeadDim + tid] = (float)acc * (1.f / kPFix);
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
    pdl_wait();   // the split pass before this kernel must have finished writing the partials
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
    return kDecodeStatusBytes + (size_t)B * Hq * nc * (kHeadDim + 2) * sizeof(float);
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
    p.status = static_cast<int *>(workspace);
    p.part_o = reinterpret_cast<float *>(static_cast<char *>(workspace) + kDecodeStatusBytes);
    p.part_ml = p.part_o + (size_t)B * Hq * p.n_chunks * kHeadDim;
    return p;
}

int launch_decode_split(const slim_cache_t *c, const void *q, const int32_t *kv_len, int B, int max_kv, int Hq,
                        float sm_scale, void *workspace, cudaStream_t stream)
{
    int C;
    const DecodeParams p = make_params(c, q, kv_len, B, max_kv, Hq, sm_scale, workspace, C);
    if (p.n_chunks == 0) return SLIM_OK;
    // SLIM_DECODE_IMPL=oneshot selects the one-block-per-chunk kernel (kept for cross-checks)
    static const bool oneshot = [] {
        const char *e = getenv("SLIM_DECODE_IMPL");
        return e != nullptr && e[0] == 'o';
    }();
    if (oneshot) return launch_decode_split_tc(p, B, stream);
    return launch_decode_split_stream(c, p, B, stream);
}

int launch_decode_merge(const slim_cache_t *c, void *out, const int32_t *kv_len, int B, int max_kv, int Hq,
                        const void *workspace, cudaStream_t stream)
{
    int C;
    const DecodeParams p = make_params(c, nullptr, kv_len, B, max_kv, Hq, 1.f, const_cast<void *>(workspace), C);
    const int rows = B * Hq;
    SLIM_CUDA_TRY(launch_pdl(slim_decode_merge_kernel, dim3((rows + 3) / 4), dim3(128), 0, stream, (const float *)p.part_o,
                             (const float *)p.part_ml, kv_len, static_cast<__nv_bfloat16 *>(out), B, Hq, p.n_chunks, C));
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
    rc = launch_decode_split(cache, q, kv_len, B, max_kv, Hq, sm_scale, scratch, (cudaStream_t)stream);
    if (rc != SLIM_OK) return rc;
    return launch_decode_merge(cache, out, kv_len, B, max_kv, Hq, scratch, (cudaStream_t)stream);
}


// Causal prefill attention over the INT8 KV cache on tcgen05 tensor cores (sm_100a).
//
// One thread block owns 128 query rows of one query head and every key they can see (the
// one-dimensional decomposition of Section 2.1: no key split, no cross-block merge).  A 128-row score
// strip over all keys does not fit on chip at long sequence lengths, so 128-key tiles stream through
// two score buffers in tensor memory with a running row maximum; the result is the same softmax
// attention.  The block is warp-specialised:
//
//   warp 8      loader: TMA tensor copies of the raw INT8 K / V tiles (128-byte swizzle) and bulk copies
//               of their scales into a 3-stage ring, completion counted on mbarriers
//   warps 4-7   dequantise in registers (the hybrid-dtype step of Section 2.2): INT8 codes -> fp16
//               code * scale / 2^e (e = the tile's largest scale exponent), written in the swizzled
//               layout the tensor cores read
//   warp 9      one thread issues tcgen05.mma: S = Q . K^T (both operands in shared memory) and
//               O += P . V (P read from tensor memory), fp32 accumulators in tensor memory
//   warps 0-3   softmax, thread = query row: tcgen05.ld of the score row, row maximum, exp2, fp16 P back
//               to tensor memory, running sum; O is rescaled only when the maximum grows by more than 2^8
//
// Scale bookkeeping per key tile: K^ = code * sk / kexp and V^ = code * sv / vexp with kexp, vexp powers of
// two, s' = acc * (kexp * row_scale) + log2(vexp), P = 2^(s' - m), O += P . V^ (the factor vexp cancels
// against 2^log2(vexp)), l += rowsum(P) / vexp.
#include <cuda.h>

#include <mutex>

#include "slim_common.cuh"
#include "slim_tcgen05.cuh"

namespace slim {

constexpr int kPtThreads = 320;
constexpr int kPtBM = 128, kPtBN = 128;
constexpr uint32_t kPtTmemCols = 512;
constexpr uint32_t kTmemS = 0, kTmemO = 256;   // S buffers at columns 0 and 128, O at 256
constexpr float kRescaleThreshold = 8.f;       // log2 units

namespace ptl {   // shared-memory map
constexpr uint32_t kQ = 0;                      // fp16 Q tile, two 64-dim halves of [128 rows][128 B]
constexpr uint32_t kKf = 32768;                 // two fp16 K tiles, same layout
constexpr uint32_t kVf = kKf + 2 * 32768;       // two fp16 V tiles: two 64-dim halves of [128 keys][128 B]
constexpr uint32_t kRaw = kVf + 2 * 32768;      // three raw stages: 16 KB INT8 tile + 512 B scales (+ pad)
constexpr uint32_t kRawStage = 17408;
constexpr uint32_t kMisc = kRaw + 3 * kRawStage;
constexpr uint32_t kBytes = kMisc + 512;
// kMisc: floats [0,2) kexp per buffer, [2,4) log2 vexp, [4,6) 1/vexp, [8,16) converter warp maxima (2 x 4);
//        byte 64: tensor-memory address; byte 128..: mbarriers
enum Bar { RAW_FULL = 0, RAW_EMPTY = 3, KF_FULL = 6, KF_EMPTY = 8, VF_FULL = 10, VF_EMPTY = 12, S_FULL = 14,
           SP_EMPTY = 16, P_FULL = 18, Q_FULL = 20, NUM_BARS = 21 };
}  // namespace ptl

struct PrefillTcParams {
    const float *scales;
    const int32_t *block_table;
    const int32_t *cu_q;
    const int32_t *kv_len;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    int *status;
    int Hq, Hkv, G, max_pages_per_seq, num_pages, n_qtiles;
    float scale_log2e;
};

__device__ __forceinline__ float fast_exp2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t hsub2_u32(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("sub.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t hmul2_u32(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("mul.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__global__ void __launch_bounds__(kPtThreads, 1)
slim_prefill_tc_kernel(const __grid_constant__ CUtensorMap codes_map, const PrefillTcParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int qtile = p.n_qtiles - 1 - blockIdx.x;   // longest rows first
    const int h = blockIdx.y, b = blockIdx.z;
    const int q0 = p.cu_q[b];
    const int q_len = p.cu_q[b + 1] - q0;
    const int m0 = qtile * kPtBM;
    if (m0 >= q_len) return;
    const int kvl = min(p.kv_len[b], p.max_pages_per_seq * kPageTokens);
    const int offset = kvl - q_len;                                   // row r sees keys j <= offset + r
    const int n_keys = min(kvl, offset + min(m0 + kPtBM, q_len));     // keys visible to the tile's last row
    const int T = n_keys > 0 ? (n_keys + kPtBN - 1) / kPtBN : 0;      // key tiles
    const int head = h / p.G;

    const uint32_t sbase = smem_u32(smem);
    float *misc_f = reinterpret_cast<float *>(smem + ptl::kMisc);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + ptl::kMisc + 64);
    const uint32_t bar0 = sbase + ptl::kMisc + 128;
    auto bar = [&](int which, int idx) { return bar0 + 8u * (uint32_t)(which + idx); };

    if (tid == 0) {
        for (int i = 0; i < 3; ++i) {
            tc::mbar_init(bar(ptl::RAW_FULL, i), 1);
            tc::mbar_init(bar(ptl::RAW_EMPTY, i), 128);
        }
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(bar(ptl::KF_FULL, i), 128);
            tc::mbar_init(bar(ptl::KF_EMPTY, i), 1);
            tc::mbar_init(bar(ptl::VF_FULL, i), 128);
            tc::mbar_init(bar(ptl::VF_EMPTY, i), 1);
            tc::mbar_init(bar(ptl::S_FULL, i), 1);
            tc::mbar_init(bar(ptl::SP_EMPTY, i), 1);
            tc::mbar_init(bar(ptl::P_FULL, i), 128);
        }
        tc::mbar_init(bar(ptl::Q_FULL, 0), 128);
        tc::mbar_init_fence();
    }
    if (warp == 9) tc::tmem_alloc(smem_u32(tmem_slot), kPtTmemCols);
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;
    auto wait = [&](uint32_t mbar, uint32_t parity) {
        if (!tc::mbar_wait(mbar, parity, ok ? (1u << 18) : 1u)) ok = false;
    };

    if (warp < 4) {
        // =========================================================== softmax: thread = query row
        const int r = tid;
        const int row = m0 + r;
        const bool row_valid = row < q_len;
        const int last_key = offset + row;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        float rs;
        {
            // Q row -> fp16 (divided by a power of two near its absmax, so the copy of bf16 is exact),
            // written as the A operand: dims [64 hf, 64 hf + 64) in half hf, 16-byte pieces XOR-swizzled by row
            uint32_t w[64];
            if (row_valid) {
                const uint4 *src = reinterpret_cast<const uint4 *>(p.q + ((size_t)(q0 + row) * p.Hq + h) * kHeadDim);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const uint4 v = __ldg(src + i);
                    w[4 * i] = v.x, w[4 * i + 1] = v.y, w[4 * i + 2] = v.z, w[4 * i + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 64; ++i) w[i] = 0u;
            }
            float am = 0.f;
#pragma unroll
            for (int i = 0; i < 64; ++i)
                am = fmaxf(am, fmaxf(fabsf(bf16_bits_to_float(w[i] & 0xFFFFu)), fabsf(bf16_bits_to_float(w[i] >> 16))));
            const float p2 = pow2_floor(am);
            const float inv = pow2_recip(p2);
            rs = p2 * p.scale_log2e;
#pragma unroll
            for (int i = 0; i < 64; ++i)
                w[i] = pack_half2(bf16_bits_to_float(w[i] & 0xFFFFu) * inv, bf16_bits_to_float(w[i] >> 16) * inv);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const uint32_t off = ptl::kQ + (uint32_t)(i >> 3) * 16384u + (uint32_t)r * 128u + (uint32_t)(((i & 7) ^ (r & 7)) << 4);
                *reinterpret_cast<uint4 *>(smem + off) = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
            }
            tc::fence_proxy_async();
            tc::mbar_arrive(bar(ptl::Q_FULL, 0));
        }

        float m_run = -INFINITY, l_run = 0.f;
        for (int j = 0; j < T; ++j) {
            const int buf = j & 1;
            wait(bar(ptl::S_FULL, buf), (j >> 1) & 1);
            __syncwarp();   // the wait loop may leave the lanes diverged; the tensor-memory ops below are warp-aligned
            tc::fence_after_sync();
            float s[128];
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t tmp[32];
                tc::tmem_ld32(tmem + lane_base + kTmemS + buf * 128 + c4 * 32, tmp);
#pragma unroll
                for (int i = 0; i < 32; ++i) s[c4 * 32 + i] = __uint_as_float(tmp[i]);
            }
            tc::tmem_ld_wait();
            const float c = fmaxf(rs * misc_f[buf], 1e-37f);   // row scale * kexp of this key tile (> 0)
            const float F = misc_f[2 + buf];              // log2 vexp
            const float vinv = misc_f[4 + buf];           // 1 / vexp
            const int key0 = j * kPtBN;
            float mx = -INFINITY;
            if (key0 + kPtBN - 1 > last_key) {
#pragma unroll
                for (int i = 0; i < 128; ++i) {
                    if (key0 + i > last_key) s[i] = -INFINITY;
                    mx = fmaxf(mx, s[i]);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 128; ++i) mx = fmaxf(mx, s[i]);
            }
            const float mt = (mx == -INFINITY) ? -INFINITY : fmaf(mx, c, F);   // c > 0: the tile's largest s'
            // the reference maximum only moves when the tile's exceeds it by more than the threshold
            const bool grow = (j == 0) ? true : (mt > m_run + kRescaleThreshold);
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
                const float alpha = grow ? fast_exp2f(m_run - mt) : 1.f;   // m_run = -inf gives 0
                wait(bar(ptl::SP_EMPTY, (j - 1) & 1), ((j - 1) >> 1) & 1);  // P.V of the previous tile is complete
                __syncwarp();
                tc::fence_after_sync();
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint32_t tmp[32];
                    tc::tmem_ld32(tmem + lane_base + kTmemO + c4 * 32, tmp);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) tmp[i] = __float_as_uint(__uint_as_float(tmp[i]) * alpha);
                    tc::tmem_st32(tmem + lane_base + kTmemO + c4 * 32, tmp);
                }
                tc::tmem_st_wait();
                l_run *= alpha;
            }
            if (grow) m_run = mt;
            const float bias = F - ((m_run == -INFINITY) ? 0.f : m_run);
            float rowsum = 0.f;
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2) {
                uint32_t pk[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float e0 = fast_exp2f(fmaf(s[c2 * 64 + 2 * i], c, bias));
                    const float e1 = fast_exp2f(fmaf(s[c2 * 64 + 2 * i + 1], c, bias));
                    rowsum += e0 + e1;
                    pk[i] = pack_half2(e0, e1);
                }
                tc::tmem_st32(tmem + lane_base + kTmemS + buf * 128 + c2 * 32, pk);
            }
            l_run = fmaf(rowsum, vinv, l_run);
            tc::tmem_st_wait();
            tc::fence_before_sync();
            tc::mbar_arrive(bar(ptl::P_FULL, buf));
        }

        // ---- epilogue: O / l -> bf16
        const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
        if (T > 0) {
            wait(bar(ptl::SP_EMPTY, (T - 1) & 1), ((T - 1) >> 1) & 1);
            __syncwarp();
            tc::fence_after_sync();
        }
        uint4 *dst = reinterpret_cast<uint4 *>(p.out + ((size_t)(q0 + row) * p.Hq + h) * kHeadDim);
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
            uint32_t tmp[32];
            if (T > 0) {
                tc::tmem_ld32(tmem + lane_base + kTmemO + c4 * 32, tmp);
                tc::tmem_ld_wait();
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) tmp[i] = 0u;
            }
            if (row_valid) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t o4[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(tmp[8 * i + 2 * k]) * inv_l,
                                                                 __uint_as_float(tmp[8 * i + 2 * k + 1]) * inv_l);
                        o4[k] = *reinterpret_cast<uint32_t *>(&v);
                    }
                    dst[c4 * 4 + i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
                }
            }
        }
    } else if (warp < 8) {
        // =========================================================== dequantise: thread = token row of the tile
        const int r = tid - 128, cw = warp - 4;
        float *cmax = misc_f + 8;
        for (int i = 0; i < 2 * T; ++i) {
            const int slot = i % 3, j = i >> 1, buf = j & 1;
            const bool is_v = (i & 1) == 0;   // V tile first, then the K tile of the same keys
            wait(bar(ptl::RAW_FULL, slot), (i / 3) & 1);
            wait(bar(is_v ? ptl::VF_EMPTY : ptl::KF_EMPTY, buf), ((j >> 1) & 1) ^ 1);
            const unsigned char *raw = smem + ptl::kRaw + slot * ptl::kRawStage;
            const int n_valid = min(kPtBN, kvl - j * kPtBN);   // rows past the cache length hold anything: zeroed
            const float sc = (r < n_valid) ? reinterpret_cast<const float *>(raw + 16384)[r] : 0.f;
            const float wm = warp_max(sc);
            if (lane == 0) cmax[(i & 1) * 4 + cw] = wm;
            tc::named_barrier(1, 128);
            const float tm = fmaxf(fmaxf(cmax[(i & 1) * 4], cmax[(i & 1) * 4 + 1]), fmaxf(cmax[(i & 1) * 4 + 2], cmax[(i & 1) * 4 + 3]));
            const float ex = pow2_floor(tm);
            const uint32_t fac2 = pack_half2(sc * pow2_recip(ex), sc * pow2_recip(ex));   // scale / 2^e in [0, 2)
            unsigned char *dstb = smem + (is_v ? ptl::kVf : ptl::kKf) + buf * 32768 + r * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 w4 = *reinterpret_cast<const uint4 *>(raw + r * 128 + ((c ^ (r & 7)) << 4));
                const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
                uint32_t hh[8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    // byte u = code ^ 0x80 under 0x64 is the fp16 number 1152 + code
                    const uint32_t x = w[k] ^ 0x80808080u;
                    hh[2 * k] = hmul2_u32(hsub2_u32(__byte_perm(x, 0x64646464u, 0x4140), 0x64806480u), fac2);
                    hh[2 * k + 1] = hmul2_u32(hsub2_u32(__byte_perm(x, 0x64646464u, 0x4342), 0x64806480u), fac2);
                }
                const uint32_t hf = (uint32_t)(c >> 2) * 16384u;
                const int oc = 2 * (c & 3);
                *reinterpret_cast<uint4 *>(dstb + hf + ((oc ^ (r & 7)) << 4)) = make_uint4(hh[0], hh[1], hh[2], hh[3]);
                *reinterpret_cast<uint4 *>(dstb + hf + (((oc + 1) ^ (r & 7)) << 4)) = make_uint4(hh[4], hh[5], hh[6], hh[7]);
            }
            if (r == 0) {
                if (is_v) {
                    misc_f[2 + buf] = (float)((int)(__float_as_uint(ex) >> 23) - 127);   // log2 of the power of two
                    misc_f[4 + buf] = pow2_recip(ex);
                } else {
                    misc_f[buf] = ex;
                }
            }
            tc::fence_proxy_async();
            tc::mbar_arrive(bar(is_v ? ptl::VF_FULL : ptl::KF_FULL, buf));
            tc::mbar_arrive(bar(ptl::RAW_EMPTY, slot));
        }
    } else if (warp == 8) {
        // =========================================================== loader (one thread)
        if (lane == 0) {
            const int32_t *bt = p.block_table + (size_t)b * p.max_pages_per_seq;
            for (int i = 0; i < 2 * T; ++i) {
                const int slot = i % 3, j = i >> 1;
                const int kv = (i & 1) ? 0 : 1;
                wait(bar(ptl::RAW_EMPTY, slot), ((i / 3) & 1) ^ 1);
                int page = bt[j];
                page = (page >= 0 && page < p.num_pages) ? page : 0;
                const uint32_t dst = sbase + ptl::kRaw + slot * ptl::kRawStage;
                const uint32_t full = bar(ptl::RAW_FULL, slot);
                tc::mbar_arrive_expect_tx(full, 16384 + 512);
                tc::tma_load_2d(dst, &codes_map, 0, ((page * p.Hkv + head) * 2 + kv) * kPageTokens, full);
                tc::bulk_load(dst + 16384, p.scales + scale_block_offset(page, head, kv, p.Hkv), 512, full);
            }
        }
    } else {
        // =========================================================== MMA issue (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc_qk = tc::instr_desc(1, 0, 0, false, false, 128, 128);   // f32 <- f16 x f16, both K-major
            constexpr uint32_t idesc_pv = tc::instr_desc(1, 0, 0, false, true, 128, 128);    // B (V) is MN-major
            auto issue_qk = [&](int j) {
                const int buf = j & 1;
                wait(bar(ptl::KF_FULL, buf), (j >> 1) & 1);
                wait(bar(ptl::SP_EMPTY, buf), ((j >> 1) & 1) ^ 1);
                tc::fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t koff = (uint32_t)(ks >> 2) * 16384u + (uint32_t)(ks & 3) * 32u;
                    const uint64_t a = tc::smem_desc(sbase + ptl::kQ + koff, 16, 1024, tc::kSwizzle128B);
                    const uint64_t bk = tc::smem_desc(sbase + ptl::kKf + buf * 32768 + koff, 16, 1024, tc::kSwizzle128B);
                    tc::mma_f16(tmem + kTmemS + buf * 128, a, bk, idesc_qk, ks > 0);
                }
                tc::commit(bar(ptl::S_FULL, buf));
                tc::commit(bar(ptl::KF_EMPTY, buf));
            };
            auto issue_pv = [&](int j) {
                const int buf = j & 1;
                wait(bar(ptl::P_FULL, buf), (j >> 1) & 1);
                wait(bar(ptl::VF_FULL, buf), (j >> 1) & 1);
                tc::fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t bv = tc::smem_desc(sbase + ptl::kVf + buf * 32768 + ks * 2048, 16384, 1024, tc::kSwizzle128B);
                    tc::mma_f16_ts(tmem + kTmemO, tmem + kTmemS + buf * 128 + ks * 8, bv, idesc_pv, (j > 0) || (ks > 0));
                }
                tc::commit(bar(ptl::VF_EMPTY, buf));
                tc::commit(bar(ptl::SP_EMPTY, buf));
            };
            wait(bar(ptl::Q_FULL, 0), 0);
            if (T > 0) issue_qk(0);
            for (int j = 0; j < T; ++j) {
                if (j + 1 < T) issue_qk(j + 1);
                issue_pv(j);
            }
        }
    }

    if (!ok && p.status != nullptr) atomicExch(p.status, SLIM_ERR_TIMEOUT);
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 9) tc::tmem_dealloc(tmem, kPtTmemCols);
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of the code pool seen as [rows][128 bytes], 128-row boxes, 128-byte swizzle.
static int codes_tensor_map(const slim_cache_t *c, CUtensorMap *out)
{
    static std::mutex mu;
    static EncodeTiledFn encode = nullptr;
    static const void *cached_ptr = nullptr;
    static long long cached_rows = 0;
    static CUtensorMap cached_map;
    std::lock_guard<std::mutex> lock(mu);
    if (encode == nullptr) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SLIM_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return SLIM_ERR_UNSUPPORTED;
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    const long long rows = (long long)c->num_pages * c->num_kv_heads * 2 * kPageTokens;
    if (cached_ptr != c->codes || cached_rows != rows) {
        const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {(cuuint64_t)kHeadDim};
        const cuuint32_t box[2] = {(cuuint32_t)kHeadDim, (cuuint32_t)kPtBN};
        const cuuint32_t estr[2] = {1, 1};
        CUresult r = encode(&cached_map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(c->codes), dims, strides,
                            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return SLIM_ERR_CUDA;
        cached_ptr = c->codes;
        cached_rows = rows;
    }
    *out = cached_map;
    return SLIM_OK;
}

size_t prefill_workspace_bytes() { return 16; }   // status word

int launch_prefill_tc(const slim_cache_t *c, const void *q, void *out, const int32_t *cu_q, const int32_t *kv_len,
                      int B, int max_q, int Hq, float sm_scale, void *workspace, cudaStream_t stream)
{
    PrefillTcParams p;
    p.scales = c->scales;
    p.block_table = c->block_table;
    p.cu_q = cu_q;
    p.kv_len = kv_len;
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.status = static_cast<int *>(workspace);
    p.Hq = Hq;
    p.Hkv = c->num_kv_heads;
    p.G = Hq / c->num_kv_heads;
    p.max_pages_per_seq = c->max_pages_per_seq;
    p.num_pages = c->num_pages;
    p.n_qtiles = (max_q + kPtBM - 1) / kPtBM;
    p.scale_log2e = sm_scale * kLog2e;
    if (p.n_qtiles == 0) return SLIM_OK;
    CUtensorMap map;
    int rc = codes_tensor_map(c, &map);
    if (rc != SLIM_OK) return rc;
    SLIM_CUDA_TRY(cudaFuncSetAttribute(slim_prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ptl::kBytes));
    dim3 grid((unsigned)p.n_qtiles, (unsigned)Hq, (unsigned)B);
    slim_prefill_tc_kernel<<<grid, kPtThreads, ptl::kBytes, stream>>>(map, p);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

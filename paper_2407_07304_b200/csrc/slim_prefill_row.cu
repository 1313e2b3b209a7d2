// SlimAttention in its literal form for short rows (sm_100a): the whole score row on chip.
//
// Section 2.1 forms every score of a block of query rows against all keys, applies one softmax to the finished
// rows and multiplies by V; nothing is ever corrected.  A 128-row block whose rows see at most 256 keys fits that
// order on this chip as it stands: the 128 x 256 fp32 score strip is 256 of the 512 tensor-memory columns, the
// output 128 more.  One thread block owns 128 query rows of one query head:
//
//   warp 4     one thread requests the raw INT8 K and V tiles (TMA, 128-byte swizzle) and their scales at once,
//              later issues the tcgen05.mma instructions
//   warps 0-3  convert the query rows to the fp16 A operand; dequantise the K tiles (thread = key row: INT8 ->
//              fp16 code * scale / 2^e, the hybrid-dtype step of Section 2.2) and, once the score MMAs have
//              read them, the V tiles into the same buffers; thread = query row for the softmax: the row's
//              maximum over all its scores first, then P = 2^(s - max) as fp16 back into tensor memory and the
//              row sum; after the P.V MMAs, O / l -> bf16.
//
// Scale bookkeeping as in the streamed kernel (slim_prefill_tc.cu): per key tile t the operands are normalised by
// the powers of two kexp(t), vexp(t) below the tile's largest K and V scale; s' = acc * kexp * row_scale + log2 vexp,
// P = 2^(s' - m) with m the maximum of s' over the whole row, O = sum_t P_t . V^_t, l = sum_t rowsum(P_t) / vexp(t).
#include <cuda.h>

#include "slim_common.cuh"
#include "slim_tcgen05.cuh"
#include "slim_tmap.cuh"

namespace slim {

constexpr int kRowThreads = 160;       // four worker warps and the warp of the loader / MMA thread
constexpr int kRowMaxKeys = 256;       // keys a block's rows may see: two 128-key tiles
constexpr uint32_t kRowTmemCols = 512; // S of tile 0 at column 0, of tile 1 at 128, O at 256 (a power of two is allocated)

namespace rwl {   // shared-memory map
constexpr uint32_t kQ = 0;                       // fp16 Q tile: two 64-dim halves of [128 rows][128 B]
constexpr uint32_t kOp = 32768;                  // two fp16 operand tiles (K^ of both key tiles, later V^), same layout
constexpr uint32_t kRaw = kOp + 2 * 32768;       // four raw stages (K0, K1, V0, V1): 16 KB INT8 tile + 512 B scales (+ pad)
constexpr uint32_t kRawStage = 17408;
constexpr uint32_t kMisc = kRaw + 4 * kRawStage; // floats [0,4): warp maxima exchange; [4,6) kexp; [6,8) log2 vexp; [8,10) 1/vexp;
                                                 // byte 64: tensor-memory address; byte 72: failure flag; byte 128..: mbarriers
constexpr uint32_t kRowScale = kMisc + 256;      // float[128]
constexpr uint32_t kBytes = kRowScale + 512;
enum Bar { RAW_FULL = 0, S_DONE = 4, O_DONE = 5, NUM_BARS = 6 };
}  // namespace rwl

struct PrefillRowParams {
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

__device__ __forceinline__ float rw_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t rw_hsub2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("sub.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t rw_hmul2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("mul.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__global__ void __launch_bounds__(kRowThreads, 1)
slim_prefill_row_kernel(const __grid_constant__ CUtensorMap codes_map, const PrefillRowParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, b = blockIdx.y, qtile = blockIdx.z;
    const int q0 = p.cu_q[b];
    const int q_len = p.cu_q[b + 1] - q0;
    const int m0 = qtile * 128;
    if (m0 >= q_len) return;
    const int kvl = min(p.kv_len[b], p.max_pages_per_seq * kPageTokens);
    const int offset = kvl - q_len;                                    // row r sees keys j <= offset + r
    const int n_keys = max(0, min(min(kvl, kRowMaxKeys), offset + min(m0 + 128, q_len)));   // (the host admits max_kv <= 256 only)
    const int T = (n_keys + 127) / 128;                                // key tiles: 0, 1 or 2
    const int head = h / p.G;

    const uint32_t sbase = smem_u32(smem);
    float *misc_f = reinterpret_cast<float *>(smem + rwl::kMisc);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + rwl::kMisc + 64);
    volatile int *fail = reinterpret_cast<volatile int *>(smem + rwl::kMisc + 72);
    const uint32_t bar0 = sbase + rwl::kMisc + 128;
    auto bar = [&](int which) { return bar0 + 8u * (uint32_t)which; };

    if (warp == 4) {
        if (lane == 0) {
            for (int i = 0; i < rwl::NUM_BARS; ++i) tc::mbar_init(bar(i), 1);
            tc::mbar_init_fence();
            *fail = 0;
            // every raw tile of the block at once: K tiles, then V tiles
            for (int i = 0; i < 2 * T; ++i) {
                const int t = i % T, kv = i / T;
                int page = __ldg(p.block_table + (size_t)b * p.max_pages_per_seq + t);
                page = (page >= 0 && page < p.num_pages) ? page : 0;
                const uint32_t dst = sbase + rwl::kRaw + (uint32_t)(kv * 2 + t) * rwl::kRawStage;
                const uint32_t full = bar(rwl::RAW_FULL + kv * 2 + t);
                tc::mbar_arrive_expect_tx(full, 16384 + 512);
                tc::tma_load_2d(dst, &codes_map, 0, ((page * p.Hkv + head) * 2 + kv) * kPageTokens, full);
                tc::bulk_load(dst + 16384, p.scales + scale_block_offset(page, head, kv, p.Hkv), 512, full);
            }
        }
        __syncwarp();
        tc::tmem_alloc(smem_u32(tmem_slot), kRowTmemCols);
    } else {
        // ---- query rows -> fp16 A operand (a row is divided by a power of two near its absmax, so the copy of bf16
        //      is exact), read coalesced: sixteen lanes per row, two rows per warp load
        float *row_scale = reinterpret_cast<float *>(smem + rwl::kRowScale);
        const int piece = lane & 15;
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
            const int rr = warp * 32 + 2 * i + (lane >> 4);
            const int row = m0 + rr;
            uint4 qv = make_uint4(0, 0, 0, 0);
            if (row < q_len) qv = __ldg(reinterpret_cast<const uint4 *>(p.q + ((size_t)(q0 + row) * p.Hq + h) * kHeadDim) + piece);
            const uint32_t w[4] = {qv.x, qv.y, qv.z, qv.w};
            float am = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                am = fmaxf(am, fmaxf(fabsf(bf16_bits_to_float(w[k] & 0xFFFFu)), fabsf(bf16_bits_to_float(w[k] >> 16))));
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
            const float p2 = pow2_floor(am);
            const float inv = pow2_recip(p2);
            uint32_t hw[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                hw[k] = pack_half2(bf16_bits_to_float(w[k] & 0xFFFFu) * inv, bf16_bits_to_float(w[k] >> 16) * inv);
            const uint32_t off = rwl::kQ + (uint32_t)(piece >> 3) * 16384u + (uint32_t)rr * 128u + (uint32_t)(((piece & 7) ^ (rr & 7)) << 4);
            *reinterpret_cast<uint4 *>(smem + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
            if (piece == 0) row_scale[rr] = p2 * p.scale_log2e;
        }
        tc::fence_proxy_async();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;
    auto wait = [&](uint32_t mbar, uint32_t parity) {
        if (!tc::mbar_wait(mbar, parity, ok ? (1u << 18) : 1u, fail)) {
            ok = false;
            *fail = 1;
        }
    };
    // INT8 -> fp16 of raw stage `stage` (thread = token row r) into operand tile `dst_tile`; returns through misc_f the
    // power of two below the tile's largest scale: [4 + t] (K) or [6 + t], [8 + t] (V: log2 and reciprocal)
    auto dequantise = [&](int stage, int dst_tile, int t, bool is_k, int n_valid) {
        const int r = tid;
        const unsigned char *raw = smem + rwl::kRaw + stage * rwl::kRawStage;
        const float sc = (r < n_valid) ? reinterpret_cast<const float *>(raw + 16384)[r] : 0.f;   // rows past the cache length hold anything: zeroed
        const float wm = warp_max(sc);
        tc::named_barrier(1, 128);          // the exchange buffer is free (its previous readers are through)
        if (lane == 0) misc_f[warp] = wm;
        tc::named_barrier(1, 128);
        const float tm = fmaxf(fmaxf(misc_f[0], misc_f[1]), fmaxf(misc_f[2], misc_f[3]));
        const float ex = (tm > 0.f) ? pow2_floor(tm) : 1.f;
        if (r == 0) {
            if (is_k) {
                misc_f[4 + t] = ex;
            } else {
                misc_f[6 + t] = (float)((int)(__float_as_uint(ex) >> 23) - 127);
                misc_f[8 + t] = pow2_recip(ex);
            }
        }
        const float f = sc * pow2_recip(ex);   // scale / 2^e in [0, 2)
        const uint32_t fac2 = pack_half2(f, f);
        unsigned char *dstb = smem + rwl::kOp + dst_tile * 32768 + r * 128;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint4 w4 = *reinterpret_cast<const uint4 *>(raw + r * 128 + ((c ^ (r & 7)) << 4));
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
            uint32_t hh[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // byte u = code ^ 0x80 under 0x64 is the fp16 number 1152 + code
                const uint32_t x = w[k] ^ 0x80808080u;
                hh[2 * k] = rw_hmul2(rw_hsub2(__byte_perm(x, 0x64646464u, 0x4140), 0x64806480u), fac2);
                hh[2 * k + 1] = rw_hmul2(rw_hsub2(__byte_perm(x, 0x64646464u, 0x4342), 0x64806480u), fac2);
            }
            const uint32_t hf = (uint32_t)(c >> 2) * 16384u;
            const int oc = 2 * (c & 3);
            *reinterpret_cast<uint4 *>(dstb + hf + ((oc ^ (r & 7)) << 4)) = make_uint4(hh[0], hh[1], hh[2], hh[3]);
            *reinterpret_cast<uint4 *>(dstb + hf + (((oc + 1) ^ (r & 7)) << 4)) = make_uint4(hh[4], hh[5], hh[6], hh[7]);
        }
    };

    float l_row = 0.f;   // softmax thread: its row's normaliser, from the softmax to the epilogue
    constexpr uint32_t idesc_qk = tc::instr_desc(1, 0, 0, false, false, 128, 128);   // f32 <- f16 x f16, both K-major
    constexpr uint32_t idesc_pv = tc::instr_desc(1, 0, 0, false, true, 128, 128);    // B (V) is MN-major
    if (warp < 4) {
        // ---- K tiles -> fp16
        for (int t = 0; t < T; ++t) {
            wait(bar(rwl::RAW_FULL + t), 0);
            dequantise(t, t, t, true, min(128, kvl - t * 128));
        }
        tc::fence_proxy_async();
    }
    tc::fence_before_sync();
    __syncthreads();                       // (1) Q and K^ operands are in place
    tc::fence_after_sync();
    if (warp == 4) {
        if (lane == 0 && T > 0) {
            // ---- every score of the block: S_t = Q . K^_t^T
            const uint64_t dq = tc::smem_desc(sbase + rwl::kQ, 16, 1024, tc::kSwizzle128B);
            for (int t = 0; t < T; ++t) {
                const uint64_t dk = tc::smem_desc(sbase + rwl::kOp + t * 32768, 16, 1024, tc::kSwizzle128B);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t koff = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
                    tc::mma_f16(tmem + (uint32_t)t * 128u, dq + koff, dk + koff, idesc_qk, ks > 0);
                }
            }
            tc::commit(bar(rwl::S_DONE));
        }
    } else if (T > 0) {
        const int r = tid;
        const int row = m0 + r;
        const int last_key = offset + row;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const float rs = reinterpret_cast<const float *>(smem + rwl::kRowScale)[r];
        wait(bar(rwl::S_DONE), 0);         // the score MMAs have read the K^ tiles: the buffers are free for V^
        __syncwarp();
        tc::fence_after_sync();
        // ---- V tiles -> fp16 (the P.V MMAs need them only after the softmax)
        for (int t = 0; t < T; ++t) {
            wait(bar(rwl::RAW_FULL + 2 + t), 0);
            dequantise(2 + t, t, t, false, min(128, kvl - t * 128));
        }
        tc::fence_proxy_async();
        tc::named_barrier(1, 128);         // every thread's kexp / vexp entries are written
        // ---- one softmax over the whole row: first the maximum of all its scores ...
        float c[2], F[2];
        float m = -INFINITY;
        for (int t = 0; t < T; ++t) {
            c[t] = fmaxf(rs * misc_f[4 + t], 1e-37f);
            F[t] = misc_f[6 + t];
            float mx = -INFINITY;
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                uint32_t v[32];
                tc::tmem_ld32(tmem + lane_base + (uint32_t)t * 128u + q4 * 32, v);
                tc::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (t * 128 + q4 * 32 + i <= last_key) mx = fmaxf(mx, __uint_as_float(v[i]));
            }
            if (mx != -INFINITY) m = fmaxf(m, fmaf(mx, c[t], F[t]));
        }
        // ---- ... then P = 2^(s' - m) as fp16 pairs into the first 64 columns of each score tile, and the row sum
        float l = 0.f;
        for (int t = 0; t < T; ++t) {
            const float bias = (m == -INFINITY) ? 0.f : F[t] - m;
            float rowsum = 0.f;
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                uint32_t v[32];
                tc::tmem_ld32(tmem + lane_base + (uint32_t)t * 128u + q4 * 32, v);
                tc::tmem_ld_wait();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int k0 = t * 128 + q4 * 32 + 2 * i;
                    const float e0 = (k0 <= last_key) ? rw_exp2(fmaf(__uint_as_float(v[2 * i]), c[t], bias)) : 0.f;
                    const float e1 = (k0 + 1 <= last_key) ? rw_exp2(fmaf(__uint_as_float(v[2 * i + 1]), c[t], bias)) : 0.f;
                    rowsum += e0 + e1;
                    pk[i] = pack_half2(e0, e1);
                }
                // (columns [16 q4, 16 q4 + 16) of the tile are overwritten; the scores still to be read lie at 32 q4 + 32 and beyond)
                tc::tmem_st16(tmem + lane_base + (uint32_t)t * 128u + q4 * 16, pk);
            }
            l = fmaf(rowsum, misc_f[8 + t], l);
        }
        tc::tmem_st_wait();
        l_row = l;
    }
    tc::fence_proxy_async();
    tc::fence_before_sync();
    __syncthreads();                       // (2) P and V^ are in place
    tc::fence_after_sync();
    if (warp == 4) {
        if (lane == 0 && T > 0) {
            // ---- O = sum_t P_t . V^_t (P read from tensor memory)
            for (int t = 0; t < T; ++t) {
                const uint64_t dv = tc::smem_desc(sbase + rwl::kOp + t * 32768, 16384, 1024, tc::kSwizzle128B);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    tc::mma_f16_ts(tmem + 256u, tmem + (uint32_t)t * 128u + ks * 8, dv + (uint64_t)((ks * 2048) >> 4), idesc_pv, t > 0 || ks > 0);
            }
            tc::commit(bar(rwl::O_DONE));
        }
    } else {
        const int r = tid;
        const int row = m0 + r;
        uint4 *dst = reinterpret_cast<uint4 *>(p.out + ((size_t)(q0 + row) * p.Hq + h) * kHeadDim);
        if (T > 0) {
            const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
            const float inv_l = (l_row > 0.f) ? 1.f / l_row : 0.f;
            wait(bar(rwl::O_DONE), 0);
            __syncwarp();
            tc::fence_after_sync();
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t v[32];
                tc::tmem_ld32(tmem + lane_base + 256u + c4 * 32, v);
                tc::tmem_ld_wait();
                if (row < q_len) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t o4[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            __nv_bfloat162 x = __floats2bfloat162_rn(__uint_as_float(v[8 * i + 2 * k]) * inv_l,
                                                                     __uint_as_float(v[8 * i + 2 * k + 1]) * inv_l);
                            o4[k] = *reinterpret_cast<uint32_t *>(&x);
                        }
                        dst[c4 * 4 + i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
                    }
                }
            }
        } else if (row < q_len) {
            // rows that see no key
#pragma unroll
            for (int i = 0; i < 16; ++i) dst[i] = make_uint4(0, 0, 0, 0);
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        if (lane == 0 && *fail != 0) {
            // a wait ran out somewhere: give the copies still in flight a bounded chance to land before the block exits
            for (int i = 0; i < 2 * T; ++i) tc::mbar_wait(bar(rwl::RAW_FULL + (i / T) * 2 + i % T), 0, 1u << 14);
            if (p.status != nullptr) atomicExch(p.status, SLIM_ERR_TIMEOUT);
        }
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(tmem, kRowTmemCols);
    }
}

// ---------------------------------------------------------------- host side
int launch_prefill_row(const slim_cache_t *c, const void *q, void *out, const int32_t *cu_q, const int32_t *kv_len,
                       int B, int max_q, int Hq, float sm_scale, void *workspace, cudaStream_t stream)
{
    PrefillRowParams p;
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
    p.n_qtiles = (max_q + 127) / 128;
    p.scale_log2e = sm_scale * kLog2e;
    if (p.n_qtiles == 0) return SLIM_OK;
    CUtensorMap map;
    int rc = codes_tensor_map(c, 128, &map);
    if (rc != SLIM_OK) return rc;
    rc = allow_dynamic_smem(reinterpret_cast<const void *>(slim_prefill_row_kernel), (int)rwl::kBytes);
    if (rc != SLIM_OK) return rc;
    if (p.n_qtiles > 65535 || B > 65535) return SLIM_ERR_UNSUPPORTED;
    dim3 grid((unsigned)Hq, (unsigned)B, (unsigned)p.n_qtiles);
    slim_prefill_row_kernel<<<grid, kRowThreads, rwl::kBytes, stream>>>(map, p);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

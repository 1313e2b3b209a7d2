// Causal prefill attention over the INT8 KV cache on tcgen05 tensor cores (sm_100a).
//
// One thread block owns 256 query rows of one query head - two 128-row tiles Q0, Q1 - and every key
// they can see (the one-dimensional decomposition of Section 2.1: no key split, no cross-block merge).
// A 256-row score strip over all keys does not fit on chip at long sequence lengths, so 128-key tiles
// stream through one score buffer per query tile in tensor memory with a running row maximum; the
// result is the same softmax attention.  Each dequantised K / V tile serves both query tiles, and
// while the softmax of one query tile runs on the ALUs the tensor cores work for the other one.
//
//   warp 12     loader: TMA tensor copies of the raw INT8 K / V tiles (128-byte swizzle) and bulk copies
//               of their scales into one raw stage for K tiles and one for V tiles, completion counted on
//               mbarriers; the tiles of the next step are prefetched into the L2 a step ahead
//   warps 8-11, 14, 15  dequantise in registers (the hybrid-dtype step of Section 2.2): INT8 codes -> fp16
//               code * scale / 2^e, written in the swizzled layout the tensor cores read.  Two K and two V
//               operand buffers: the converters run a key tile ahead of the tensor cores (with one buffer each
//               the conversion of V(j) and K(j+1) sat between P.V(j-1) and Q.K(j+1)^T on the critical path).
//               A thread of warps 8-11 owns a token row and converts six of its eight 16-code pieces, the
//               two spare warps of the last warp group take the other two pieces of every row
//   warp 13     one thread issues tcgen05.mma in the order  P0.V(j), Q0.K(j+1)^T, P1.V(j), Q1.K(j+1)^T:
//               S_t = Q_t . K^T (both operands in shared memory), O_t += P_t . V (P read from tensor
//               memory), fp32 accumulators in tensor memory
//   warps 0-3   softmax of Q0, warps 4-7 softmax of Q1; thread = query row.  The whole 128-column score row is
//               read into registers with one tcgen05.ld round trip (the softmax warps take registers from the
//               other warp groups: setmaxnreg), then row maximum, exp2 -> fp16 P back to tensor memory and the
//               running sum.  O is rescaled only when the maximum grows by more than 2^8.
//
// Scale bookkeeping per key tile j: K^ = code * sk / kexp(j) and V^ = code * sv / vexp(j) with kexp(j), vexp(j)
// the powers of two below the tile's largest K / V scale, so both operands stay in [0, 2) * 127 whatever the
// magnitudes; s' = acc * (kexp * row_scale) + log2 vexp, P = 2^(s' - m), O += P . V^ (the factor vexp cancels
// against 2^log2(vexp)), l += rowsum(P) / vexp, out = O / l.  vexp(j) is published as soon as the raw V tile has
// landed (before its conversion), so the softmax of tile j never waits for it in practice.
#include <cuda.h>

#include "slim_common.cuh"
#include "slim_tcgen05.cuh"
#include "slim_tmap.cuh"

namespace slim {

constexpr int kPfThreads = 512;   // four warp groups: softmax 0, softmax 1, dequantisers, {loader, MMA thread, two idle warps}
constexpr int kPfBM = 128, kPfBN = 128;
constexpr int kPfRows = 2 * kPfBM;             // query rows per block
constexpr int kPfRawStages = 2;                // one raw stage for K tiles, one for V tiles
constexpr int kPfConvWarps = 6;                // warps 8-11 and the two spare warps of the last warp group
constexpr uint32_t kPfTmemCols = 512;
constexpr uint32_t kPfTmemS = 0, kPfTmemO = 256;   // S_t at columns 128 t, O_t at 256 + 128 t
constexpr float kPfRescaleThreshold = 8.f;     // log2 units

namespace pfl {   // shared-memory map
constexpr uint32_t kQ = 0;                      // two fp16 Q tiles; a tile = two 64-dim halves of [128 rows][128 B]
constexpr uint32_t kKf = 65536;                 // two fp16 K tiles (key tiles j even / odd), same layout
constexpr uint32_t kVf = kKf + 2 * 32768;       // two fp16 V tiles: two 64-dim halves of [128 keys][128 B] each
constexpr uint32_t kRaw = kVf + 2 * 32768;      // raw INT8 tiles: stage 0 K, stage 1 V (16 KB each, 1 KB aligned for the swizzle)
constexpr uint32_t kRawScales = kRaw + kPfRawStages * 16384;   // their scales, 512 B per stage
constexpr uint32_t kMisc = kRawScales + kPfRawStages * 512;
constexpr uint32_t kRowScale = kMisc + 512;     // float[2][128]: row scale of every query row (written by the thread that converts the row)
constexpr uint32_t kBytes = kRowScale + 1024;
// kMisc: floats by the key tile's position j mod 4: [0,4) kexp, [4,8) log2 vexp, [8,12) 1 / vexp;
//        byte 64: tensor-memory address; byte 72: failure flag; byte 128..: mbarriers
enum Bar { RAW_FULL = 0, RAW_EMPTY = 2, KF_FULL = 4, KF_EMPTY = 6, VF_FULL = 8, VF_EMPTY = 10,
           S_FULL = 12, P_FULL = 14, O_DONE = 16, Q_FULL = 18, VEXP_FULL = 20, NUM_BARS = 24 };
static_assert(128 + 8 * NUM_BARS <= 512, "mbarriers fit the misc area");
static_assert(kBytes <= 232448, "shared memory budget of one block");
}  // namespace pfl

struct PrefillTcParams {
    const float *scales;
    const int32_t *block_table;
    const int32_t *cu_q;
    const int32_t *kv_len;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    int *status;
    int Hq, Hkv, G, max_pages_per_seq, num_pages, n_qblocks;
    float scale_log2e;
};

__device__ __forceinline__ float pf_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
// packed fp32 pairs in a 64-bit register (two values per instruction)
__device__ __forceinline__ uint64_t pf_pack(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void pf_unpack(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;\n" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t pf_fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t pf_add2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float pf_max3(float a, float b, float c)
{
    float m;
    asm("max.f32 %0, %1, %2, %3;\n" : "=f"(m) : "f"(a), "f"(b), "f"(c));
    return m;
}
__device__ __forceinline__ uint32_t pf_hsub2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("sub.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t pf_hmul2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("mul.rn.f16x2 %0, %1, %2;\n" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// kTwoPass: the literal order of Section 2.1 - every score of a row before its softmax.  The block walks its key
// tiles twice: the first pass only takes the row maxima of the scores, the second computes P = 2^(s - max) against
// that final maximum and accumulates P.V, so no accumulator is ever corrected.  Both passes run through the same
// pipeline (a key tile is loaded and converted again in the second pass); the tile sequence of the block is
// simply twice as long, and barrier phases count positions in that sequence.
template <bool kTwoPass>
__global__ void __launch_bounds__(kPfThreads, 1)
slim_prefill_tc_kernel(const __grid_constant__ CUtensorMap codes_map, const PrefillTcParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Blocks are handed out in the order of their linear index: heads vary fastest, then sequences, then row
    // blocks from the last (which sees the most keys) to the first, so that the longest blocks of every head and
    // sequence start first and the short ones fill the tail of the launch.
    const int qblock = p.n_qblocks - 1 - blockIdx.z;
    const int h = blockIdx.x, b = blockIdx.y;
    const int q0 = p.cu_q[b];
    const int q_len = p.cu_q[b + 1] - q0;
    const int m0 = qblock * kPfRows;
    if (m0 >= q_len) return;
    const int kvl = min(p.kv_len[b], p.max_pages_per_seq * kPageTokens);
    const int offset = kvl - q_len;                                   // row r sees keys j <= offset + r
    // key tiles of the two query tiles: tile t covers rows [m0 + 128 t, m0 + 128 t + 128)
    int Tt[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int first = m0 + t * kPfBM;
        const int n_keys = (first < q_len) ? min(kvl, offset + min(first + kPfBM, q_len)) : 0;
        Tt[t] = n_keys > 0 ? (n_keys + kPfBN - 1) / kPfBN : 0;
    }
    const int T0 = Tt[0], T1 = Tt[1];
    const int T = max(T0, T1);
    const int NT = kTwoPass ? 2 * T : T;   // positions in the block's tile sequence
    const int head = h / p.G;

    const uint32_t sbase = smem_u32(smem);
    float *misc_f = reinterpret_cast<float *>(smem + pfl::kMisc);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + pfl::kMisc + 64);
    volatile int *fail = reinterpret_cast<volatile int *>(smem + pfl::kMisc + 72);
    const uint32_t bar0 = sbase + pfl::kMisc + 128;
    auto bar = [&](int which, int idx) { return bar0 + 8u * (uint32_t)(which + idx); };

    // The first global-memory round trips of the block start before its set-up is complete: the loader thread
    // initialises the ring's "full" barriers itself and requests the first raw tiles at once, and the softmax
    // threads read their query rows into registers; both overlap the barrier set-up and the tensor-memory allocation.
    int raw_issued = 0;   // loader thread: raw tiles requested so far
    int page_next = 0;
    auto request_raw = [&](int i) {
        const int32_t *bt = p.block_table + (size_t)b * p.max_pages_per_seq;
        const int kv = i & 1, j = i >> 1;   // K tiles go through raw stage 0, V tiles through stage 1
        int page = page_next;
        page = (page >= 0 && page < p.num_pages) ? page : 0;
        const uint32_t full = bar(pfl::RAW_FULL, kv);
        tc::mbar_arrive_expect_tx(full, 16384 + 512);
        tc::tma_load_2d(sbase + pfl::kRaw + kv * 16384, &codes_map, 0, ((page * p.Hkv + head) * 2 + kv) * kPageTokens, full);
        tc::bulk_load(sbase + pfl::kRawScales + kv * 512, p.scales + scale_block_offset(page, head, kv, p.Hkv), 512, full);
        if (kv == 1 && j + 1 < NT) {
            // the next key tile's page id, and its two tiles on their way into the L2 a step before they are asked for
            page_next = __ldg(bt + ((kTwoPass && j + 1 >= T) ? j + 1 - T : j + 1));
            const int pn = (page_next >= 0 && page_next < p.num_pages) ? page_next : 0;
            tc::tma_prefetch_2d(&codes_map, 0, ((pn * p.Hkv + head) * 2) * kPageTokens);
            tc::tma_prefetch_2d(&codes_map, 0, ((pn * p.Hkv + head) * 2 + 1) * kPageTokens);
        }
        ++raw_issued;
    };
    if (warp == 12 && lane == 0) {
        for (int i = 0; i < kPfRawStages; ++i) tc::mbar_init(bar(pfl::RAW_FULL, i), 1);
        tc::mbar_init_fence();
        // everything above, and the other warps' set-up and query rows, may overlap the end of the kernel before
        // this one in the stream (the append of the one-call prefill step); the cache is read from here on
        pdl_wait();
        if (T > 0) {
            page_next = __ldg(p.block_table + (size_t)b * p.max_pages_per_seq);
            for (int i = 0; i < min(kPfRawStages, 2 * NT); ++i) request_raw(i);   // every stage is free the first time round
        }
    }
    // Query rows are read coalesced: sixteen lanes read one row's 256 bytes, so a warp's load covers two whole rows
    // (a thread per row would touch 32 rows with 16 bytes each, and the load/store unit would be busy with those
    // scattered sectors for microseconds while the set-up's own shared-memory traffic queues behind them).  A warp
    // of query tile t converts the tile's rows 32 (warp & 3) + 2 i + (lane >> 4), i = 0..15; a lane holds piece
    // lane & 15 (eight dims) of each.
    uint4 qv[16];
    if (warp < 8) {
        const int t = warp >> 2;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int rr = (warp & 3) * 32 + 2 * i + (lane >> 4);
            const int row = m0 + t * kPfBM + rr;
            qv[i] = make_uint4(0, 0, 0, 0);
            if (Tt[t] > 0 && row < q_len)
                qv[i] = __ldg(reinterpret_cast<const uint4 *>(p.q + ((size_t)(q0 + row) * p.Hq + h) * kHeadDim) + (lane & 15));
        }
    }

    if (tid == 0) {
        for (int t = 0; t < 2; ++t) {
            tc::mbar_init(bar(pfl::RAW_EMPTY, t), kPfConvWarps);   // (one arrival per converter warp)
            tc::mbar_init(bar(pfl::KF_FULL, t), kPfConvWarps);
            tc::mbar_init(bar(pfl::KF_EMPTY, t), 1);
            tc::mbar_init(bar(pfl::VF_FULL, t), kPfConvWarps);
            tc::mbar_init(bar(pfl::VF_EMPTY, t), 1);
            tc::mbar_init(bar(pfl::S_FULL, t), 1);
            tc::mbar_init(bar(pfl::P_FULL, t), 128);
            tc::mbar_init(bar(pfl::O_DONE, t), 1);
            tc::mbar_init(bar(pfl::Q_FULL, t), 128);
        }
        for (int i = 0; i < 4; ++i) tc::mbar_init(bar(pfl::VEXP_FULL, i), 1);
        tc::mbar_init_fence();
        *fail = 0;
    }
    if (warp == 13) tc::tmem_alloc(smem_u32(tmem_slot), kPfTmemCols);
    if (warp < 8 && Tt[warp >> 2] > 0) {
        // (needs nothing of the set-up: it overlaps the barrier initialisation and the tensor-memory allocation)
        const int t = warp >> 2;
        // Q rows -> fp16 (a row is divided by a power of two near its absmax, so the copy of bf16 is exact),
        // written as the A operand: dims [64 hf, 64 hf + 64) in half hf, 16-byte pieces XOR-swizzled by row
        float *row_scale = reinterpret_cast<float *>(smem + pfl::kRowScale) + t * kPfBM;
        const int piece = lane & 15;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int rr = (warp & 3) * 32 + 2 * i + (lane >> 4);
            const uint32_t w[4] = {qv[i].x, qv[i].y, qv[i].z, qv[i].w};
            float am = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                am = fmaxf(am, fmaxf(fabsf(bf16_bits_to_float(w[k] & 0xFFFFu)), fabsf(bf16_bits_to_float(w[k] >> 16))));
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));   // the row's sixteen lanes
            const float p2 = pow2_floor(am);
            const float inv = pow2_recip(p2);
            uint32_t hw[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                hw[k] = pack_half2(bf16_bits_to_float(w[k] & 0xFFFFu) * inv, bf16_bits_to_float(w[k] >> 16) * inv);
            const uint32_t off = pfl::kQ + (uint32_t)t * 32768u + (uint32_t)(piece >> 3) * 16384u + (uint32_t)rr * 128u +
                                 (uint32_t)(((piece & 7) ^ (rr & 7)) << 4);
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
    // Registers move from the warp groups that need few to the softmax groups, which hold a whole 128-column
    // score row (every warp of a group executes the same setmaxnreg; 2 * 160 + 96 + 96 = 4 * 128 per lane; the split was chosen by measurement).
    if (warp < 8) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 160;\n");
    } else if (warp < 12) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 96;\n");
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 96;\n");
    }

    if (warp < 8) {
        // =========================================================== softmax of query tile t: thread = query row
        const int t = warp >> 2;
        const int r = tid & 127;
        const int row = m0 + t * kPfBM + r;
        const bool row_valid = row < q_len;
        const int last_key = offset + row;
        const int Tmine = t ? T1 : T0;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_base + kPfTmemS + (uint32_t)t * 128u;
        const uint32_t tO = tmem + lane_base + kPfTmemO + (uint32_t)t * 128u;
        float rs = 0.f;
        if (Tmine > 0) {
            // the tile's rows were converted before the set-up's barrier, which also ordered the row scales
            tc::mbar_arrive(bar(pfl::Q_FULL, t));
            rs = reinterpret_cast<const float *>(smem + pfl::kRowScale)[t * kPfBM + r];
        }

        float m_run = -INFINITY, l_run = 0.f;
        const int steps = kTwoPass ? 2 * Tmine : Tmine;   // this query tile's steps (its count of S_FULL / P_FULL / O_DONE phases)
        for (int jj = 0; jj < steps; ++jj) {
            const bool second = kTwoPass && jj >= Tmine;
            const int j = second ? jj - Tmine : jj;       // key tile
            const int jv = second ? T + j : j;            // its position in the block's tile sequence
            wait(bar(pfl::S_FULL, t), (uint32_t)jj & 1u);
            __syncwarp();   // the wait loop may leave the lanes diverged; the tensor-memory ops below are warp-aligned
            tc::fence_after_sync();
            wait(bar(pfl::VEXP_FULL, jv & 3), (uint32_t)(jv >> 2) & 1u);   // published long before, as a rule
            const float c = fmaxf(rs * misc_f[jv & 3], 1e-37f);   // row scale * kexp of this key tile (> 0)
            const float F = misc_f[4 + (jv & 3)];                 // log2 vexp
            const float vinv = misc_f[8 + (jv & 3)];              // 1 / vexp
            const int key0 = j * kPfBN;
            const bool diag = key0 + kPfBN - 1 > last_key;       // some of this tile's keys are masked for this row
            // ---- the whole score row into registers with one round trip to tensor memory, then its maximum
            //      (c > 0, so the maximum of the raw accumulators commutes with the scaling)
            uint32_t v[128];
            {
                uint32_t(&v0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&v[0]);
                uint32_t(&v1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&v[32]);
                uint32_t(&v2)[32] = *reinterpret_cast<uint32_t(*)[32]>(&v[64]);
                uint32_t(&v3)[32] = *reinterpret_cast<uint32_t(*)[32]>(&v[96]);
                tc::tmem_ld32(tS, v0);
                tc::tmem_ld32(tS + 32, v1);
                tc::tmem_ld32(tS + 64, v2);
                tc::tmem_ld32(tS + 96, v3);
                tc::tmem_ld_wait();
            }
            // causal mask: only warps that touch the diagonal execute it (minus infinity becomes weight 0 below)
            if (__any_sync(0xffffffffu, diag)) {
#pragma unroll
                for (int i = 0; i < 128; ++i)
                    if (key0 + i > last_key) v[i] = 0xFF800000u;
            }
            float mx = -INFINITY, mx2 = -INFINITY;   // two chains
#pragma unroll
            for (int i = 0; i < 128; i += 4) {
                mx = pf_max3(mx, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                mx2 = pf_max3(mx2, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
            }
            mx = fmaxf(mx, mx2);
            const float mt = (mx == -INFINITY) ? -INFINITY : fmaf(mx, c, F);   // the tile's largest s'
            if (kTwoPass && !second) {
                // first pass: the row's maximum only; the score buffer is free for the next tile's scores
                m_run = fmaxf(m_run, mt);
                tc::fence_before_sync();
                tc::mbar_arrive(bar(pfl::P_FULL, t));
                continue;
            }
            // the reference maximum only moves when the tile's exceeds it by more than the threshold
            // (second pass of the two-pass form: it is the row's final maximum and never moves)
            const bool grow = kTwoPass ? false : ((j == 0) ? true : (mt > m_run + kPfRescaleThreshold));
            if (!kTwoPass && j > 0 && __any_sync(0xffffffffu, grow)) {
                const float alpha = grow ? pf_exp2(m_run - mt) : 1.f;   // m_run = -inf gives 0
                wait(bar(pfl::O_DONE, t), (uint32_t)(j - 1) & 1u);      // P.V of the previous tile is complete
                __syncwarp();
                tc::fence_after_sync();
#pragma unroll 1
                for (int k = 0; k < 8; ++k) {
                    uint32_t v[16];
                    tc::tmem_ld16(tO + k * 16, v);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                    tc::tmem_st16(tO + k * 16, v);
                }
                tc::tmem_st_wait();
                l_run *= alpha;
            }
            if (grow) m_run = mt;
            const float bias = (m_run == -INFINITY) ? 0.f : F - m_run;
            // ---- P = 2^(s - m) as fp16 pairs, packed in place, into the first 64 columns of the score buffer
            // (packed fp32 arithmetic: one fused multiply-add and one add per pair of scores)
            const uint64_t c2 = pf_pack(c, c), bias2 = pf_pack(bias, bias);
            uint64_t sum2a = 0ull, sum2b = 0ull;
#pragma unroll
            for (int i = 0; i < 64; ++i) {
                float x0, x1;
                pf_unpack(pf_fma2(pf_pack(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])), c2, bias2), x0, x1);
                const float e0 = pf_exp2(x0), e1 = pf_exp2(x1);
                if (i & 1) sum2b = pf_add2(sum2b, pf_pack(e0, e1)); else sum2a = pf_add2(sum2a, pf_pack(e0, e1));
                v[i] = pack_half2(e0, e1);
            }
            float rowsum, rowsum_hi;
            pf_unpack(pf_add2(sum2a, sum2b), rowsum, rowsum_hi);
            rowsum += rowsum_hi;
            {
                const uint32_t(&p0)[32] = *reinterpret_cast<const uint32_t(*)[32]>(&v[0]);
                const uint32_t(&p1)[32] = *reinterpret_cast<const uint32_t(*)[32]>(&v[32]);
                tc::tmem_st32(tS, p0);
                tc::tmem_st32(tS + 32, p1);
            }
            l_run = fmaf(rowsum, vinv, l_run);
            tc::tmem_st_wait();
            tc::fence_before_sync();
            tc::mbar_arrive(bar(pfl::P_FULL, t));
        }

        // ---- epilogue: O / l -> bf16
        if (Tmine > 0) {
            wait(bar(pfl::O_DONE, t), (uint32_t)(steps - 1) & 1u);
            __syncwarp();
            tc::fence_after_sync();
            const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
            // The rows go out coalesced: every thread puts its bf16 row into the tile's Q buffer (no score MMA of this
            // block reads it any more), 16-byte piece i of row r rotated to piece slot (i + r) mod 16 so that neither
            // these stores nor the loads below collide on banks; then sixteen lanes write one row's 256 bytes, two rows
            // per warp store.  A warp reads back only rows its own threads wrote.
            unsigned char *stage = smem + pfl::kQ + (uint32_t)t * 32768u;
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t v[32];
                tc::tmem_ld32(tO + c4 * 32, v);
                tc::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t o4[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        __nv_bfloat162 x = __floats2bfloat162_rn(__uint_as_float(v[8 * i + 2 * k]) * inv_l,
                                                                 __uint_as_float(v[8 * i + 2 * k + 1]) * inv_l);
                        o4[k] = *reinterpret_cast<uint32_t *>(&x);
                    }
                    *reinterpret_cast<uint4 *>(stage + r * 256 + (((c4 * 4 + i + r) & 15) << 4)) = make_uint4(o4[0], o4[1], o4[2], o4[3]);
                }
            }
            __syncwarp();
            const int piece = lane & 15;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int rr = (warp & 3) * 32 + 2 * i + (lane >> 4);
                const int orow = m0 + t * kPfBM + rr;
                const uint4 o = *reinterpret_cast<const uint4 *>(stage + rr * 256 + (((piece + rr) & 15) << 4));
                if (orow < q_len)
                    reinterpret_cast<uint4 *>(p.out + ((size_t)(q0 + orow) * p.Hq + h) * kHeadDim)[piece] = o;
            }
        } else if (row_valid) {
            // a row that sees no key
            uint4 *dst = reinterpret_cast<uint4 *>(p.out + ((size_t)(q0 + row) * p.Hq + h) * kHeadDim);
#pragma unroll
            for (int i = 0; i < 16; ++i) dst[i] = make_uint4(0, 0, 0, 0);
        }
    } else if (warp < 12 || warp >= 14) {
        // =========================================================== dequantise
        // A thread of warps 8-11 owns token row r = tid - 256 of every tile and converts its pieces 0..5 (a piece =
        // 16 codes); a thread of warps 14, 15 owns rows u and u + 64 (u = tid - 448) and converts their pieces 6, 7
        // (consecutive lanes on consecutive rows: the swizzled 16-byte slots of a warp's access then cover all banks).
        const bool main_cv = warp < 12;
        const int r0 = main_cv ? tid - 256 : tid - 448;
        const int n_rows = main_cv ? 1 : 2, c_first = main_cv ? 0 : 6, c_last = main_cv ? 6 : 8;
        const bool announces = warp == 8 && lane == 0;   // the thread that publishes a tile's exponents
        for (int i = 0; i < 2 * NT; ++i) {
            const int kv = i & 1, j = i >> 1;   // j: position in the block's tile sequence; K tile first, then the V tile of the same keys
            const bool is_k = kv == 0;
            const int buf = j & 1;
            wait(bar(pfl::RAW_FULL, kv), (uint32_t)j & 1u);
            const unsigned char *raw = smem + pfl::kRaw + kv * 16384;
            const float *scales = reinterpret_cast<const float *>(smem + pfl::kRawScales + kv * 512);
            const int n_valid = min(kPfBN, kvl - ((kTwoPass && j >= T) ? j - T : j) * kPfBN);   // rows past the cache length hold anything: zeroed
            // power of two below the tile's largest scale (every warp finds it for itself: four scales per lane)
            float wm = 0.f;
            {
                const float4 s4 = *reinterpret_cast<const float4 *>(scales + 4 * lane);
                const float sv[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (4 * lane + k < n_valid) wm = fmaxf(wm, sv[k]);
                wm = warp_max(wm);
            }
            const float ex = (wm > 0.f) ? pow2_floor(wm) : 1.f;
            const float rex = pow2_recip(ex);
            if (is_k) {
                if (announces) misc_f[j & 3] = ex;
                wait(bar(pfl::KF_EMPTY, buf), ((uint32_t)(j >> 1) & 1u) ^ 1u);
            } else {
                // the softmax of this key tile needs the V exponent before the V tile itself is converted
                if (announces) {
                    misc_f[4 + (j & 3)] = (float)((int)(__float_as_uint(ex) >> 23) - 127);   // log2 of the power of two
                    misc_f[8 + (j & 3)] = rex;
                    tc::mbar_arrive(bar(pfl::VEXP_FULL, j & 3));
                }
                wait(bar(pfl::VF_EMPTY, buf), ((uint32_t)(j >> 1) & 1u) ^ 1u);
            }
            unsigned char *dst_tile = smem + (is_k ? pfl::kKf : pfl::kVf) + buf * 32768;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (q >= n_rows) break;
                const int r = r0 + 64 * q;
                const float f = ((r < n_valid) ? scales[r] : 0.f) * rex;   // scale / 2^e in [0, 2)
                const uint32_t fac2 = pack_half2(f, f);
                unsigned char *dstb = dst_tile + r * 128;
                for (int c = c_first; c < c_last; ++c) {
                    const uint4 w4 = *reinterpret_cast<const uint4 *>(raw + r * 128 + ((c ^ (r & 7)) << 4));
                    const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
                    uint32_t hh[8];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        // byte u = code ^ 0x80 under 0x64 is the fp16 number 1152 + code
                        const uint32_t x = w[k] ^ 0x80808080u;
                        hh[2 * k] = pf_hmul2(pf_hsub2(__byte_perm(x, 0x64646464u, 0x4140), 0x64806480u), fac2);
                        hh[2 * k + 1] = pf_hmul2(pf_hsub2(__byte_perm(x, 0x64646464u, 0x4342), 0x64806480u), fac2);
                    }
                    const uint32_t hf = (uint32_t)(c >> 2) * 16384u;
                    const int oc = 2 * (c & 3);
                    *reinterpret_cast<uint4 *>(dstb + hf + ((oc ^ (r & 7)) << 4)) = make_uint4(hh[0], hh[1], hh[2], hh[3]);
                    *reinterpret_cast<uint4 *>(dstb + hf + (((oc + 1) ^ (r & 7)) << 4)) = make_uint4(hh[4], hh[5], hh[6], hh[7]);
                }
            }
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                tc::mbar_arrive(bar(is_k ? pfl::KF_FULL : pfl::VF_FULL, buf));
                tc::mbar_arrive(bar(pfl::RAW_EMPTY, kv));
            }
        }
    } else if (warp == 12) {
        // =========================================================== loader (one thread)
        if (lane == 0 && T > 0) {
            for (int i = kPfRawStages; i < 2 * NT; ++i) {   // the first K and V tile were requested during set-up
                wait(bar(pfl::RAW_EMPTY, i & 1), ((uint32_t)(i >> 1) & 1u) ^ 1u);
                request_raw(i);
            }
        }
    } else if (warp == 13) {
        // =========================================================== MMA issue (one thread)
        if (lane == 0 && T > 0) {
            constexpr uint32_t idesc_qk = tc::instr_desc(1, 0, 0, false, false, 128, 128);   // f32 <- f16 x f16, both K-major
            constexpr uint32_t idesc_pv = tc::instr_desc(1, 0, 0, false, true, 128, 128);    // B (V) is MN-major
            // Operand descriptors are built once; an MMA step only adds a constant to the address field.
            const uint64_t dq0 = tc::smem_desc(sbase + pfl::kQ, 16, 1024, tc::kSwizzle128B);
            const uint64_t dq1 = tc::smem_desc(sbase + pfl::kQ + 32768u, 16, 1024, tc::kSwizzle128B);
            const uint64_t dk0 = tc::smem_desc(sbase + pfl::kKf, 16, 1024, tc::kSwizzle128B);      // K^ buffer 0; buffer 1 lies 32 KB behind it
            const uint64_t dv0 = tc::smem_desc(sbase + pfl::kVf, 16384, 1024, tc::kSwizzle128B);
            auto issue_qk = [&](int t, int buf) {   // S_t = Q_t . K^T
                const uint64_t dq = t ? dq1 : dq0;
                const uint64_t dk = dk0 + (uint64_t)(buf * (32768 >> 4));
                const uint32_t d = tmem + kPfTmemS + (uint32_t)t * 128u;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    // dims [16 ks, 16 ks + 16): half ks / 4 of the tile (16 KB apart), 32 bytes per step inside the swizzle span
                    const uint64_t koff = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
                    tc::mma_f16(d, dq + koff, dk + koff, idesc_qk, ks > 0);
                }
                tc::commit(bar(pfl::S_FULL, t));
            };
            auto issue_pv = [&](int t, bool first, int buf) {   // O_t (+)= P_t . V
                const uint32_t d = tmem + kPfTmemO + (uint32_t)t * 128u, a = tmem + kPfTmemS + (uint32_t)t * 128u;
                const uint64_t dv = dv0 + (uint64_t)(buf * (32768 >> 4));
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)   // keys [16 ks, 16 ks + 16): 2 KB further down the V tile, 8 columns of P
                    tc::mma_f16_ts(d, a + ks * 8, dv + (uint64_t)((ks * 2048) >> 4), idesc_pv, !first || ks > 0);
                tc::commit(bar(pfl::O_DONE, t));
            };
            if (T0 > 0) wait(bar(pfl::Q_FULL, 0), 0);
            if (T1 > 0) wait(bar(pfl::Q_FULL, 1), 0);
            wait(bar(pfl::KF_FULL, 0), 0);
            tc::fence_after_sync();
            if (T0 > 0) issue_qk(0, 0);
            if (T1 > 0) issue_qk(1, 0);
            tc::commit(bar(pfl::KF_EMPTY, 0));
            // The fixed order P0.V(j), Q0.K(j+1)^T, P1.V(j), Q1.K(j+1)^T keeps the two query tiles half a step
            // apart, so that their softmax phases (which share the special-function units) alternate.
            int c0 = 0, c1 = 0;   // two-pass form: steps each query tile has taken (its barrier phases)
            for (int jv = 0; jv < NT; ++jv) {
                const uint32_t ph = (uint32_t)jv & 1u;                       // parity of the query tiles' barriers at this position
                const int buf = jv & 1, bufn = buf ^ 1;                      // operand buffers of this position's V tile / the next one's K tile
                const uint32_t bph = (uint32_t)(jv >> 1) & 1u, bphn = (uint32_t)((jv + 1) >> 1) & 1u;   // parities of those buffers' barriers
                const bool second = kTwoPass && jv >= T;
                const int j = second ? jv - T : jv;                          // key tile at this position
                const int jn = (kTwoPass && jv + 1 >= T) ? jv + 1 - T : jv + 1;   // key tile at the next position
                const bool more = jv + 1 < NT;
                const bool a0 = j < T0, a1 = j < T1, n0 = more && jn < T0, n1 = more && jn < T1;
                const bool pv = !kTwoPass || second;                         // the first pass has no P.V
                wait(bar(pfl::VF_FULL, buf), bph);
                if (a0) {
                    wait(bar(pfl::P_FULL, 0), kTwoPass ? ((uint32_t)c0 & 1u) : ph);
                    tc::fence_after_sync();
                    if (pv) issue_pv(0, j == 0, buf); else tc::commit(bar(pfl::O_DONE, 0));
                    ++c0;
                }
                if (n0 || n1) wait(bar(pfl::KF_FULL, bufn), bphn);
                if (n0) {
                    tc::fence_after_sync();
                    issue_qk(0, bufn);
                }
                if (a1) {
                    wait(bar(pfl::P_FULL, 1), kTwoPass ? ((uint32_t)c1 & 1u) : ph);
                    tc::fence_after_sync();
                    if (pv) issue_pv(1, j == 0, buf); else tc::commit(bar(pfl::O_DONE, 1));
                    ++c1;
                }
                tc::commit(bar(pfl::VF_EMPTY, buf));
                if (n1) {
                    tc::fence_after_sync();
                    issue_qk(1, bufn);
                }
                if (n0 || n1) tc::commit(bar(pfl::KF_EMPTY, bufn));
            }
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    if (warp == 12 && lane == 0 && *fail != 0) {
        // a wait ran out somewhere: give the copies still in flight a bounded chance to land before the block exits
        for (int i = max(0, raw_issued - kPfRawStages); i < raw_issued; ++i)
            tc::mbar_wait(bar(pfl::RAW_FULL, i & 1), (uint32_t)(i >> 1) & 1u, 1u << 14);
        if (p.status != nullptr) atomicExch(p.status, SLIM_ERR_TIMEOUT);
    }
    if (warp == 13) {
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(tmem, kPfTmemCols);
    }
}

// ---------------------------------------------------------------- host side
size_t prefill_workspace_bytes() { return 16; }   // status word

int launch_prefill_tc(const slim_cache_t *c, const void *q, void *out, const int32_t *cu_q, const int32_t *kv_len,
                      int B, int max_q, int Hq, float sm_scale, void *workspace, cudaStream_t stream, bool two_pass, bool after_append)
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
    p.n_qblocks = (max_q + kPfRows - 1) / kPfRows;
    p.scale_log2e = sm_scale * kLog2e;
    if (p.n_qblocks == 0) return SLIM_OK;
    CUtensorMap map;
    int rc = codes_tensor_map(c, kPfBN, &map);
    if (rc != SLIM_OK) return rc;
    rc = allow_dynamic_smem(two_pass ? reinterpret_cast<const void *>(slim_prefill_tc_kernel<true>)
                                     : reinterpret_cast<const void *>(slim_prefill_tc_kernel<false>), (int)pfl::kBytes);
    if (rc != SLIM_OK) return rc;
    if (p.n_qblocks > 65535 || B > 65535) return SLIM_ERR_UNSUPPORTED;
    dim3 grid((unsigned)Hq, (unsigned)B, (unsigned)p.n_qblocks);
    if (two_pass) slim_prefill_tc_kernel<true><<<grid, kPfThreads, pfl::kBytes, stream>>>(map, p);
    else if (after_append) SLIM_CUDA_TRY(launch_pdl(slim_prefill_tc_kernel<false>, grid, dim3(kPfThreads), pfl::kBytes, stream, map, p));
    else slim_prefill_tc_kernel<false><<<grid, kPfThreads, pfl::kBytes, stream>>>(map, p);
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

}  // namespace slim

// Decode split pass as a persistent streaming kernel (sm_100a): TMA ring -> tcgen05 -> partials.
//
// The next-token phase is bound by memory bandwidth (Section 2.2, Eq. 1: every cached byte is read once
// per generated token).  The kernel therefore keeps the copy engine busy all the time and spends almost
// no instructions per cached byte:
//
//  * One thread block per SM.  The work - every 256-token chunk of every (sequence, kv head) - is cut
//    into one contiguous range per block.  A chunk is the unit of a partial result (m, l, O[128]).
//  * Two producer threads, each in a warp of its own, walk the block's chunks: one asks the TMA engine
//    for each chunk's INT8 K tiles and V tiles into a ring of 16 KB tile stages (128-byte swizzled,
//    completion counted on mbarriers), the other for its scales and query rows into a small ring of
//    chunk records (one thread hands the copy engine about one request per 100 ns, which alone would
//    limit the stream).  Their two warps also find the block's range, one its start and one its end.  A
//    stage goes back to the producer the moment the tensor cores have read it (the MMA completion
//    itself arrives on the stage's mbarrier), so K tiles are held only until the scores are out and
//    most of the ring is in flight at any time.  A ragged last tile is fetched in 16-row boxes so
//    that no byte beyond the chunk's tokens (rounded up to 16) is read.
//  * One more warp per consumer group holds that group's MMA-issuing thread: it waits for the chunk's
//    tiles and for the group's operands, issues the tcgen05.mma instructions and commits their
//    completion to the group's mbarrier and to the stages' "empty" mbarriers.
//  * Three consumer groups of four warps (two when a kv head serves more than eight query heads) take
//    chunks in turn.  For its chunk a group
//      - builds the query operand: a 22-bit fixed-point copy of the G = Hq/Hkv query rows of the kv
//        head, three signed bytes per value (columns [high | middle | low bytes]), so that a row with a
//        few channels hundreds of times larger than the rest keeps the small channels' precision;
//      - S^T[token][head] = K_codes . Q^T by tcgen05.mma kind::i8: the INT8 codes are the operand as
//        they are (the hybrid-dtype step of Section 2.2 happens inside the tensor core);
//      - one softmax over the chunk's 256 scores per head (Section 2.1 order: all scores, softmax,
//        then .V), thread = token, after a tensor-memory load;
//      - O^T[dim][head] = V_codes^T . P^T, again kind::i8, V read MN-major straight from its
//        token-major rows, P as 16-bit fixed point in two unsigned bytes;
//      - recombines the byte planes and writes the partial.
//    While one group computes, the other groups' chunks and the next chunks are in flight.
//  * The chunks cover every token of a sequence but the last one.  The last token is attended from registers by
//    one consumer warp while the first tiles are on their way: its K and V rows come either from the caller
//    (one-call step: the warp quantises them and stores them in the cache) or from the cache, and the warp
//    writes the token's own partial (m, l, O) into the slot after the row's last chunk.  A decode step whose
//    new token starts a chunk of its own therefore costs no chunk, and nothing in the kernel reads a cache row
//    that the kernel itself wrote.
//
// The V scale is folded into the softmax weight (s'_j = s_j + log2 sv_j, P_j = 2^(s'_j - max s'),
// o = sum P_j c_j / sum P_j / sv_j), so P <= 1 is normalised by the chunk's largest contribution.
// Every wait is bounded; a wait that runs out raises the status word and the block drains and exits.
#include <cuda.h>

#include "slim_common.cuh"
#include "slim_decode_params.cuh"
#include "slim_quant.cuh"
#include "slim_tcgen05.cuh"
#include "slim_tmap.cuh"

namespace slim {

constexpr int kStGroupThreads = 128;
constexpr int kStTile = 128;                                    // tokens per MMA tile (= one page)
constexpr int kStChunk = 2 * kStTile;                           // tokens per chunk / partial
constexpr int kStTailBox = 16;                                  // rows per TMA box of a ragged tile
constexpr uint32_t kStTileBytes = kStTile * kHeadDim;           // 16 KB
constexpr float kStQFix = 1048576.f;   // 2^20: |q / pow2| < 2  ->  |v| < 2^21: bytes [hi in [-32, 32] | mid | lo]
constexpr float kStPFix = 65535.f;

static_assert(kStChunk == 256, "partials are indexed by 256-token chunks (decode_workspace_bytes, merge kernel)");

template <int NH, bool kAppend = false>
struct StSmem {
    static constexpr int NS = (3 * NH + 15) / 16 * 16;      // score MMA columns: [hi | mid | lo bytes of NH heads], padded to 16
    static constexpr int NP = 2 * NH;                       // output MMA columns: [hi | lo bytes of P for NH heads]
    static constexpr int kGroups = (NH <= 8) ? 3 : 2;       // consumer groups (chunks in process at a time)
    static constexpr int kThreads = kGroups * kStGroupThreads + 64 + kGroups * 32;   // groups + two producer warps + one MMA-issue warp per group
    static constexpr int kProducerWarp = kGroups * 4;
    static constexpr int kInfoSlots = 2 * kGroups;          // chunk records in flight
    static constexpr uint32_t kTmemCols = (kGroups <= 2) ? 256 : 512;   // 128 per group: S of two tiles + O
    static_assert(2 * NS + NP <= 128, "a group's accumulators fit its 128 tensor-memory columns");
    static constexpr int kStages = (NH <= 8) ? 10 : 9;      // tile stages of the ring
    // chunk record: both scale vectors, the kv head's query rows, the chunk's coordinates
    static constexpr uint32_t kScales = 0;                  // per tile: 128 K scales, then 128 V scales
    static constexpr uint32_t kQraw = 2048;                 // bf16 [G][128]
    static constexpr uint32_t kMeta = kQraw + NH * 256;     // int[5]: sequence, kv head, chunk, valid tokens, first tile index
    static constexpr uint32_t kInfoBytes = (kMeta + 32 + 127) / 128 * 128;
    static constexpr uint32_t kInfo0 = kStages * kStTileBytes;
    // per consumer group
    static constexpr uint32_t kGroup0 = kInfo0 + kInfoSlots * kInfoBytes;
    static constexpr uint32_t kPTileBytes = NP * 128;       // a P^T tile, core-matrix layout
    static constexpr uint32_t kP = 0;                       // two P^T tiles
    static constexpr uint32_t kQop = 2 * kPTileBytes;       // query operand: NS rows x 128 bytes, core-matrix layout
    static constexpr uint32_t kLsum = kQop + NS * 128;      // floats [NH][128]: every token thread's share of the softmax denominators
    static constexpr uint32_t kRed = kLsum + NH * 512;      // floats: [NH][4] warp maxima, [NH] row scales
    static constexpr uint32_t kGroupBytes = (kRed + 5 * NH * 4 + 127) / 128 * 128;
    // block-wide: mbarriers full[kStages], empty[kStages], info full[4], info empty[4],
    //             operands ready for S[2], for PV[2], S done[2], PV done[2]
    static constexpr uint32_t kBar = kGroup0 + kGroups * kGroupBytes;
    static constexpr int kNumBars = 2 * kStages + 2 * kInfoSlots + 4 * kGroups;
    static constexpr uint32_t kTmemSlot = kBar + kNumBars * 8;
    static constexpr uint32_t kRange = (kTmemSlot + 8 + 15) / 16 * 16;   // int[6]: -, the block's first sequence / head / chunk, that sequence's chunks and chunk tokens; at +32: long long[2], the global chunk indices where the range starts and ends
    static constexpr uint32_t kFail = kRange + 48;
    static constexpr uint32_t kBytes = kFail + 16;
    static_assert(kRange % 16 == 0, "range record is read as int4-aligned ints");
    static_assert(kBytes <= 232448, "shared memory budget of one block");
};

// Byte offset of element (row n, k byte kb) of a K-major operand stored as 8x16-byte core matrices:
// 16 bytes of k contiguous, 8 rows 16 bytes apart, next 16 k-bytes +128, next 8 rows +1024.
__device__ __forceinline__ uint32_t st_core_off(int n, int kb)
{
    return (uint32_t)((n >> 3) * 1024 + (kb >> 4) * 128 + (n & 7) * 16 + (kb & 15));
}

__device__ __forceinline__ float st_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float st_rcp(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
// Order-preserving map between floats and signed integers (its own inverse), so that an integer
// warp reduction finds a floating-point maximum.
__device__ __forceinline__ int st_ordered_int(float x)
{
    const int i = __float_as_int(x);
    return i ^ ((i >> 31) & 0x7FFFFFFF);
}
__device__ __forceinline__ float st_ordered_float(int i)
{
    return __int_as_float(i ^ ((i >> 31) & 0x7FFFFFFF));
}

// A sequence's cached tokens, never beyond the page table or the launch's max_kv.
__device__ __forceinline__ int st_clamped_len(const DecodeParams &p, int b)
{
    const int cap = min(p.max_pages_per_seq * kPageTokens, p.n_chunks * kStChunk);
    return min(max(__ldg(p.kv_len + b), 0), cap);
}

// The tokens of a sequence that the chunks cover: all but the last one, which is attended from registers.
__device__ __forceinline__ int st_chunk_len(const DecodeParams &p, int b)
{
    return max(st_clamped_len(p, b) - 1, 0);
}

// Steps (sequence, kv head, chunk) to the next chunk in the order the work is cut in; sequences without
// chunks are skipped.  Only called while another chunk exists, so a sequence with chunks is always found.
__device__ __forceinline__ void st_next_chunk(const DecodeParams &p, int B, int &b, int &head, int &chunk, int &len, int &nc)
{
    if (++chunk == nc) {
        chunk = 0;
        if (++head == p.Hkv) {
            head = 0;
            do {
                ++b;
                len = (b < B) ? st_chunk_len(p, b) : kStChunk;   // b < B always holds inside a block's range
                nc = (len + kStChunk - 1) / kStChunk;
            } while (nc == 0);
        }
    }
}

// floor(a / b) for 0 <= a, 0 < b: the 64-bit division is only taken when the dividend needs it
__device__ __forceinline__ long long st_div(long long a, int b)
{
    if (((unsigned long long)a >> 32) == 0ull) return (long long)((unsigned)a / (unsigned)b);
    return a / b;
}

// The last token of (sequence b, kv head `head`), at position L - 1, attended by one warp from registers
// (lanes 0-15 hold its K row, lanes 16-31 its V row, eight dims per lane).  With kAppend and a length that was
// not clamped the rows are the caller's new token: they are quantised here and stored in the cache (Section
// 2.2; exactly the codes and scales slim_kv_append writes); otherwise they are read from the cache.  For each
// of the G query heads the token's partial - score s' = s + log2(sv), weight P = 1, so m = s', l = 1 / sv and
// O = the V codes - goes to slot `slot` of the row; with to_out (a sequence of one token in a launch that merges
// its own partials) the result code * sv is written straight to the output instead.
template <bool kAppend>
__device__ __forceinline__ void st_last_token(const DecodeParams &p, int b, int head, int L, int slot, int lane, bool to_out)
{
    const int kv = lane >> 4, l = lane & 15;
    const int pos = L - 1;
    const int page_raw = __ldg(p.block_table + (size_t)b * p.max_pages_per_seq + (pos >> 7));
    const bool page_ok = page_raw >= 0 && page_raw < p.num_pages;
    const int page = page_ok ? page_raw : 0;
    const int row_in_page = pos & (kPageTokens - 1);
    const size_t code_off = code_block_offset(page, head, kv, p.Hkv) + (size_t)row_in_page * kHeadDim;
    const size_t scale_off = scale_block_offset(page, head, kv, p.Hkv) + row_in_page;
    uint2 pk;
    float scale;
    if (kAppend && __ldg(p.kv_len + b) == L) {   // (the same for every lane of the warp)
        const __nv_bfloat16 *src = (kv ? p.v_new : p.k_new) + ((size_t)b * p.Hkv + head) * kHeadDim;
        pk = quantize_row16(__ldg(reinterpret_cast<const uint4 *>(src) + l), scale);
        if (page_ok) {
            reinterpret_cast<uint2 *>(const_cast<int8_t *>(p.codes) + code_off)[l] = pk;
            if (l == 0) const_cast<float *>(p.scales)[scale_off] = scale;
        }
    } else {
        pk = __ldg(reinterpret_cast<const uint2 *>(p.codes + code_off) + l);
        scale = __ldg(p.scales + scale_off);
    }
    const float sk = __shfl_sync(0xffffffffu, scale, 0);
    const float sv = fmaxf(__shfl_sync(0xffffffffu, scale, 16), kMinScale);
    float c[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        c[i] = (float)(int)(int8_t)((pk.x >> (8 * i)) & 0xFFu);
        c[4 + i] = (float)(int)(int8_t)((pk.y >> (8 * i)) & 0xFFu);
    }
    const float lsv = __log2f(sv), rsv = st_rcp(sv), ks = sk * p.scale_log2e;
    if (to_out) {
        // a sequence of one token: its softmax weight is 1 and the result is the dequantised V row
        if (kv == 1) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                __nv_bfloat162 x = __floats2bfloat162_rn(c[2 * i] * sv, c[2 * i + 1] * sv);
                w[i] = *reinterpret_cast<uint32_t *>(&x);
            }
            for (int h = 0; h < p.G; ++h)
                reinterpret_cast<uint4 *>(p.out + ((size_t)b * p.Hq + (size_t)head * p.G + h) * kHeadDim)[l] = make_uint4(w[0], w[1], w[2], w[3]);
        }
        return;
    }
    const size_t row0 = (size_t)b * p.Hq + (size_t)head * p.G;
    for (int h0 = 0; h0 < p.G; h0 += 8) {
        // eight heads' query rows are requested together (one round trip instead of eight)
        uint4 qv[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            qv[i] = (h0 + i < p.G) ? __ldg(reinterpret_cast<const uint4 *>(p.q + (row0 + h0 + i) * kHeadDim) + l) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (h0 + i >= p.G) break;
            const uint32_t qw[4] = {qv[i].x, qv[i].y, qv[i].z, qv[i].w};
            float dot = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                dot = fmaf(bf16_bits_to_float(qw[k] & 0xFFFFu), c[2 * k], dot);
                dot = fmaf(bf16_bits_to_float(qw[k] >> 16), c[2 * k + 1], dot);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);   // lanes 0-15: q . k codes
            const float s = __shfl_sync(0xffffffffu, dot, 0);
            const size_t ps = (row0 + h0 + i) * p.n_slots + slot;
            if (kv == 1) {
                float4 *dst = reinterpret_cast<float4 *>(p.part_o + ps * kHeadDim + 8 * l);
                dst[0] = make_float4(c[0], c[1], c[2], c[3]);
                dst[1] = make_float4(c[4], c[5], c[6], c[7]);
            }
            if (lane == 0) *reinterpret_cast<float2 *>(p.part_ml + ps * 2) = make_float2(fmaf(s, ks, lsv), rsv);
        }
    }
}

// Log-sum-exp merge of the nc partials (the chunks' and the last token's) of the G query heads of (sequence b, kv head `head`) by one warp:
//   M = max m_c;  l = sum l_c 2^(m_c - M);  o = sum O_c 2^(m_c - M) / l   (a lane owns four head dims).
// The caller has made sure that every partial of the pair is visible; they are read past the L1 cache.
__device__ __forceinline__ void st_merge_rows(const DecodeParams &p, int b, int head, int nc, int lane)
{
    constexpr int kBatch = 12;   // partial outputs requested before the first of them is used
    for (int h = 0; h < p.G; ++h) {
        const size_t row = (size_t)b * p.Hq + (size_t)head * p.G + h;
        const float2 *ml = reinterpret_cast<const float2 *>(p.part_ml) + row * p.n_slots;
        const float4 *po = reinterpret_cast<const float4 *>(p.part_o + row * p.n_slots * kHeadDim) + lane;
        // every load of the first round is in flight before anything waits for one of them
        float4 o[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) o[u] = (u < nc) ? __ldcg(po + (size_t)u * (kHeadDim / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float2 first = (lane < nc) ? __ldcg(ml + lane) : make_float2(-INFINITY, 0.f);
        float M = first.x;
        for (int c = lane + 32; c < nc; c += 32) M = fmaxf(M, __ldcg(ml + c).x);
        M = warp_max(M);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l = 0.f;
        for (int c0 = 0; c0 < nc; c0 += 32) {
            float w = 0.f;   // stays 0 for the lanes past the last chunk
            if (c0 + lane < nc) {
                const float2 v = (c0 == 0) ? first : __ldcg(ml + c0 + lane);
                w = exp2f(v.x - M);
                l = fmaf(v.y, w, l);
            }
            for (int j0 = 0; j0 < min(32, nc - c0); j0 += kBatch) {
                if (c0 + j0 > 0) {
#pragma unroll
                    for (int u = 0; u < kBatch; ++u)
                        o[u] = (j0 + u < 32 && c0 + j0 + u < nc) ? __ldcg(po + (size_t)(c0 + j0 + u) * (kHeadDim / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const float wj = __shfl_sync(0xffffffffu, w, (j0 + u) & 31);
                    acc.x = fmaf(o[u].x, wj, acc.x);
                    acc.y = fmaf(o[u].y, wj, acc.y);
                    acc.z = fmaf(o[u].z, wj, acc.z);
                    acc.w = fmaf(o[u].w, wj, acc.w);
                }
            }
        }
        l = warp_sum(l);
        const float inv = (l > 0.f) ? 1.f / l : 0.f;
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t *>(&lo);
        packed.y = *reinterpret_cast<uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(p.out + row * kHeadDim + lane * 4) = packed;
    }
}

template <int NH, bool kAppend, bool kMerge>
__global__ void __launch_bounds__(StSmem<NH, kAppend>::kThreads, 1)
slim_decode_stream_kernel(const __grid_constant__ CUtensorMap map_tile, const __grid_constant__ CUtensorMap map_tail,
                          const DecodeParams p, const int B)
{
    using L = StSmem<NH, kAppend>;
    constexpr int NS = L::NS, NP = L::NP;
    constexpr int S = L::kStages;
    constexpr int kStGroups = L::kGroups, kStInfoSlots = L::kInfoSlots;
    constexpr int kPW = L::kProducerWarp;
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::kBar;
    auto bar_full = [&](int st) { return bar0 + 8u * (uint32_t)st; };
    auto bar_empty = [&](int st) { return bar0 + 8u * (uint32_t)(S + st); };
    auto bar_info_full = [&](int i) { return bar0 + 8u * (uint32_t)(2 * S + i); };
    auto bar_info_empty = [&](int i) { return bar0 + 8u * (uint32_t)(2 * S + kStInfoSlots + i); };
    auto bar_ready_s = [&](int g) { return bar0 + 8u * (uint32_t)(2 * S + 2 * kStInfoSlots + g); };
    auto bar_ready_pv = [&](int g) { return bar0 + 8u * (uint32_t)(2 * S + 2 * kStInfoSlots + kStGroups + g); };
    auto bar_mma_s = [&](int g) { return bar0 + 8u * (uint32_t)(2 * S + 2 * kStInfoSlots + 2 * kStGroups + g); };
    auto bar_mma_pv = [&](int g) { return bar0 + 8u * (uint32_t)(2 * S + 2 * kStInfoSlots + 3 * kStGroups + g); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::kTmemSlot);
    int *range = reinterpret_cast<int *>(smem + L::kRange);
    volatile int *fail = reinterpret_cast<volatile int *>(smem + L::kFail);

    pdl_launch_dependents();   // the merge kernel queued behind this one may be scheduled; it waits for our completion

    // ---- the producers' walk over the block's chunk list.  State of one walker (each producer thread has its own):
    int w_b = 0, w_head = 0, w_chunk = 0, w_len = 0, w_nc = 1;   // the chunk the walker stands on
    int2 w_pg = make_int2(0, 0);                                  // its two page ids (requested one chunk ahead)
    int tiles_issued = 0;                                         // tile stages of the chunks walked so far (ring position)
    bool ok = true;
    auto wait = [&](uint32_t mbar, uint32_t parity) {
        if (!tc::mbar_wait(mbar, parity, ok ? (1u << 18) : 1u, fail)) {
            ok = false;
            *fail = 1;
        }
    };
    auto page_ids = [&](int bb, int cc) {
        const int32_t *bt = p.block_table + (size_t)bb * p.max_pages_per_seq + cc * 2;
        int2 r;
        r.x = (cc * 2 < p.max_pages_per_seq) ? __ldg(bt) : 0;
        r.y = (cc * 2 + 1 < p.max_pages_per_seq) ? __ldg(bt + 1) : 0;
        return r;
    };
    const uint64_t stream_policy = tc::policy_evict_first();   // cache rows are read once per launch
    auto walk_begin = [&]() {
        w_b = range[1], w_head = range[2], w_chunk = range[3], w_nc = range[4], w_len = range[5];
        w_pg = page_ids(w_b, w_chunk);
    };
    // Walks chunks [n_from, n_to) of the block's list, asking the copy engine for each chunk's tiles (K tiles, then V
    // tiles, in the order the consumers need them) and / or for its record: coordinates, the scales of its tiles (K
    // and V scales of a page and head are adjacent: one 1 KB copy per tile) and the query rows unless the group that
    // takes the chunk still holds them from its previous chunk (same sequence and kv head).
    auto walk = [&](int n_from, int n_to, int n_end, bool tiles, bool records) {
        for (int n = n_from; n < n_to; ++n) {
            const int cb = w_b, chead = w_head, cchunk = w_chunk;
            const int n_tok = min(kStChunk, w_len - w_chunk * kStChunk);
            const int2 cpg = w_pg;
            // ---- the next chunk's coordinates and page ids, requested before this chunk's copies are issued
            if (n + 1 < n_end) {
                st_next_chunk(p, B, w_b, w_head, w_chunk, w_len, w_nc);
                w_pg = page_ids(min(w_b, B - 1), w_chunk);
            }
            int page[2] = {cpg.x, cpg.y};
            int rows16[2];
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                page[t] = (page[t] >= 0 && page[t] < p.num_pages) ? page[t] : 0;
                const int rows = max(0, min(kStTile, n_tok - t * kStTile));
                rows16[t] = (rows + kStTailBox - 1) / kStTailBox * kStTailBox;
            }
            const int n_tiles = rows16[1] > 0 ? 2 : 1;
            if (records) {
                const int islot = n % kStInfoSlots;
                const uint32_t iph = (uint32_t)(n / kStInfoSlots) & 1u;
                wait(bar_info_empty(islot), iph ^ 1u);
                unsigned char *info = smem + L::kInfo0 + islot * L::kInfoBytes;
                const uint32_t info_addr = sbase + L::kInfo0 + islot * L::kInfoBytes;
                int *meta = reinterpret_cast<int *>(info + L::kMeta);
                meta[0] = cb, meta[1] = chead, meta[2] = cchunk, meta[3] = n_tok, meta[4] = tiles_issued;
                const bool need_q = !(n >= kStGroups && cchunk >= kStGroups);
                const uint32_t q_bytes = need_q ? (uint32_t)p.G * kHeadDim * 2u : 0u;
                tc::mbar_arrive_expect_tx(bar_info_full(islot), (uint32_t)n_tiles * 1024u + q_bytes);
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    if (t < n_tiles)
                        tc::bulk_load(info_addr + L::kScales + t * 1024, p.scales + scale_block_offset(page[t], chead, 0, p.Hkv),
                                      1024u, bar_info_full(islot));
                if (need_q)
                    tc::bulk_load(info_addr + L::kQraw, p.q + ((size_t)cb * p.Hq + (size_t)chead * p.G) * kHeadDim, q_bytes,
                                  bar_info_full(islot));
            }
            if (tiles) {
                int gi = tiles_issued;
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (rows16[t] == 0) continue;
                        const int stage = gi % S;
                        wait(bar_empty(stage), ((uint32_t)(gi / S) & 1u) ^ 1u);
                        const uint32_t full = bar_full(stage);
                        tc::mbar_arrive_expect_tx(full, (uint32_t)rows16[t] * kHeadDim);
                        const int row0 = ((page[t] * p.Hkv + chead) * 2 + kv) * kPageTokens;
                        const uint32_t dst = sbase + (uint32_t)stage * kStTileBytes;
                        if (rows16[t] == kStTile) {
                            tc::tma_load_2d_hint(dst, &map_tile, 0, row0, full, stream_policy);
                        } else {
                            for (int r = 0; r < rows16[t]; r += kStTailBox)
                                tc::tma_load_2d_hint(dst + r * kHeadDim, &map_tail, 0, row0 + r, full, stream_policy);
                        }
                        ++gi;
                    }
                }
            }
            tiles_issued += 2 * n_tiles;
        }
    };
    constexpr int kBarSetup = 8, kBarProducers = 9;   // named barriers (1 .. kGroups belong to the consumer groups)

    if (warp == kPW && lane == 0) {
        tc::prefetch_tensormap(&map_tile);   // (kernel parameters: nothing an earlier kernel writes)
        tc::prefetch_tensormap(&map_tail);
        for (int i = 0; i < S; ++i) {
            tc::mbar_init(bar_full(i), 1);
            tc::mbar_init(bar_empty(i), 1);
        }
        for (int i = 0; i < kStInfoSlots; ++i) {
            tc::mbar_init(bar_info_full(i), 1);
            // a chunk record is released by the 128 threads of its group and that group's MMA thread
            tc::mbar_init(bar_info_empty(i), kStGroupThreads + 1);
        }
        for (int g = 0; g < kStGroups; ++g) {
            tc::mbar_init(bar_ready_s(g), kStGroupThreads);
            tc::mbar_init(bar_ready_pv(g), kStGroupThreads);
            tc::mbar_init(bar_mma_s(g), 1);
            tc::mbar_init(bar_mma_pv(g), 1);
        }
        tc::mbar_init_fence();
        *fail = 0;
    }
    if (warp == kPW) tc::tmem_alloc(smem_u32(tmem_slot), L::kTmemCols);
    if (warp == kPW || warp == kPW + 1) {
        // Up to here the block may run beside the kernel before it in the stream (the same step's
        // slim_kv_append); from here on it reads what earlier kernels may have written.
        pdl_wait();
        // ---- this block's contiguous range of chunks, in (sequence, kv head, chunk) order.  The work is cut
        //      by 128-token tiles (what a chunk costs) and the cut points are moved up to chunk starts.  The first
        //      producer warp finds where the range starts, the second where it ends, at the same time.
        // The cut at tile index x (x <= total tiles): the number of chunks that start before it, over all (sequence,
        // kv head) runs in order, and where it falls: sequence, kv head, chunk (which may be the run's chunk count:
        // the cut then lies at the start of the next run), that sequence's chunk count and chunk tokens.
        struct Cut {
            long long index;
            int b, head, chunk, nc, len;
        };
        Cut cut;
        cut.b = cut.head = cut.chunk = cut.len = 0;
        cut.nc = 1;
        const int which = warp - kPW;   // 0: the range's start, 1: its end
        const int len_first = (lane < B) ? st_chunk_len(p, lane) : 0;   // tokens of the first 32 sequences that chunks cover
        const int len_u = __shfl_sync(0xffffffffu, len_first, 0);
        bool uniform = __all_sync(0xffffffffu, lane >= B || len_first == len_u);
        for (int base = 32; base < B && uniform; base += 32)
            uniform = __all_sync(0xffffffffu, base + lane >= B || st_chunk_len(p, base + lane) == len_u);
        if (uniform) {
            // every sequence has the same length (a batch decoded in lockstep): the cut has a closed form
            const int nt = (len_u + kStTile - 1) / kStTile, nc = (len_u + kStChunk - 1) / kStChunk;
            const long long pairs = (long long)B * p.Hkv;
            const long long x = st_div(pairs * nt * (blockIdx.x + which), (int)gridDim.x);
            cut.index = pairs * nc;
            if (x < pairs * nt) {
                const long long pair = st_div(x, nt);
                const int d = (int)(x - pair * nt);
                cut.b = (int)st_div(pair, p.Hkv);
                cut.head = (int)(pair - (long long)cut.b * p.Hkv);
                cut.chunk = min(nc, (d + 1) / 2);
                cut.nc = nc;
                cut.len = len_u;
                cut.index = pair * nc + cut.chunk;
            }
        } else {
            // a warp scan over the sequences' tile and chunk counts, 32 sequences at a time
            struct Scan {
                int len, nt, nc, it, ic;   // tokens covered by chunks, tiles, chunks; inclusive prefix sums of tiles and chunks over the lanes
            };
            auto scan_block = [&](int base) {
                Scan r;
                const int b = base + lane;
                r.len = (base == 0) ? len_first : ((b < B) ? st_chunk_len(p, b) : 0);
                r.nt = (r.len + kStTile - 1) / kStTile;
                r.nc = (r.len + kStChunk - 1) / kStChunk;
                r.it = r.nt;
                r.ic = r.nc;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int vt = __shfl_up_sync(0xffffffffu, r.it, o), vc = __shfl_up_sync(0xffffffffu, r.ic, o);
                    if (lane >= o) r.it += vt, r.ic += vc;
                }
                return r;
            };
            const Scan first = scan_block(0);
            long long tiles_all = __shfl_sync(0xffffffffu, first.it, 31);
            for (int base = 32; base < B; base += 32) tiles_all += __shfl_sync(0xffffffffu, scan_block(base).it, 31);
            const long long x = st_div(tiles_all * p.Hkv * (blockIdx.x + which), (int)gridDim.x);
            long long tiles_pre = 0, chunks_pre = 0;
            bool found = false;
            for (int base = 0; base < B && !found; base += 32) {
                const Scan sc = (base == 0) ? first : scan_block(base);
                const unsigned hit = __ballot_sync(0xffffffffu, (tiles_pre + sc.it) * p.Hkv > x);
                if (hit != 0u) {
                    const int l = __ffs(hit) - 1;
                    const int nt_l = __shfl_sync(0xffffffffu, sc.nt, l), nc_l = __shfl_sync(0xffffffffu, sc.nc, l);
                    const long long tb = tiles_pre + __shfl_sync(0xffffffffu, sc.it, l) - nt_l;
                    const long long cb = chunks_pre + __shfl_sync(0xffffffffu, sc.ic, l) - nc_l;
                    const int r = (int)(x - tb * p.Hkv);             // < Hkv * nt_l
                    const int head = r / nt_l, d = r - head * nt_l;
                    cut.b = base + l;
                    cut.head = head;
                    cut.chunk = min(nc_l, (d + 1) / 2);
                    cut.nc = nc_l;
                    cut.len = __shfl_sync(0xffffffffu, sc.len, l);
                    cut.index = cb * p.Hkv + (long long)head * nc_l + cut.chunk;
                    found = true;
                } else {
                    tiles_pre += __shfl_sync(0xffffffffu, sc.it, 31);
                    chunks_pre += __shfl_sync(0xffffffffu, sc.ic, 31);
                }
            }
            if (!found) cut.index = chunks_pre * p.Hkv;
        }
        long long *cut_index = reinterpret_cast<long long *>(smem + L::kRange + 32);
        if (lane == 0) {
            cut_index[which] = cut.index;
            if (which == 0) {
                // one step from the chunk before the cut: a cut at the end of a run moves to the next run with chunks
                int b0 = cut.b, head0 = cut.head, chunk0 = cut.chunk - 1, nc0 = cut.nc, len0 = cut.len;
                st_next_chunk(p, B, b0, head0, chunk0, len0, nc0);
                range[1] = min(b0, B - 1);   // (beyond the last sequence only when the range is empty)
                range[2] = head0;
                range[3] = chunk0;
                range[4] = nc0;
                range[5] = len0;
            }
        }
        // the two warps exchange what they found
        __threadfence_block();
        tc::named_barrier(kBarProducers, 64);
    } else if (warp < kPW) {
        // rows of the query operand that belong to no head stay zero for the whole launch
        const int g = warp >> 2, gtid = tid & 127;
        unsigned char *qop = smem + L::kGroup0 + g * L::kGroupBytes + L::kQop;
        for (int i = gtid * 16; i < NS * 128; i += kStGroupThreads * 16) *reinterpret_cast<uint4 *>(qop + i) = make_uint4(0, 0, 0, 0);
    }
    // ---- the block's set-up barrier.  The two producer warps do not wait on it (they have exchanged the range through
    //      a barrier of their own): they signal their arrival and start asking for the first chunks at once, so that
    //      those copies are in flight while the other warps are still on their way.
    tc::fence_proxy_async();
    tc::fence_before_sync();
    __threadfence_block();
    if (warp == kPW || warp == kPW + 1) {
        tc::named_barrier_arrive(kBarSetup, L::kThreads);
    } else {
        tc::named_barrier(kBarSetup, L::kThreads);
    }
    tc::fence_after_sync();
    const uint32_t tmem = (warp == kPW || warp == kPW + 1) ? 0u : *tmem_slot;   // (the producers do not touch tensor memory)
    const long long *cut_index_all = reinterpret_cast<const long long *>(smem + L::kRange + 32);
    const int cnt = (int)(cut_index_all[1] - cut_index_all[0]);

    if (warp == kPW || warp == kPW + 1) {
        // =========================================================== producers (one thread each)
        // warp kPW walks the block's chunks and asks for their K and V tiles; warp kPW + 1 walks the same list and
        // asks for the chunk records.  Two threads because the rate at which one thread can hand requests to the
        // copy engine (about one per 100 ns) would otherwise limit the stream.
        if (lane == 0 && cnt > 0) {
            walk_begin();
            walk(0, cnt, cnt, warp == kPW, warp == kPW + 1);
        }
    } else if (warp > kPW + 1) {
        // =========================================================== MMA issue for group g (one thread)
        const int g = warp - kPW - 2;
        if (lane == 0) {
            const uint32_t grp_addr = sbase + L::kGroup0 + g * L::kGroupBytes;
            const uint32_t tm = tmem + (uint32_t)g * 128u;
            constexpr uint32_t idesc_s = tc::instr_desc(2, 1, 1, false, false, 128, NS);   // s32 <- s8 (K-major) x s8 (K-major)
            constexpr uint32_t idesc_pv = tc::instr_desc(2, 1, 0, true, false, 128, NP);   // s32 <- s8 (MN-major) x u8 (K-major)
            // operand descriptors are built once; an MMA step only adds a constant to the address field
            const uint64_t dk0 = tc::smem_desc(sbase, 16, 1024, tc::kSwizzle128B);         // a K tile in stage 0
            const uint64_t dv0 = tc::smem_desc(sbase, 1024, 1024, tc::kSwizzle128B);       // a V tile in stage 0 (MN-major)
            const uint64_t dq = tc::smem_desc(grp_addr + L::kQop, 128, 1024, tc::kSwizzleNone);
            const uint64_t dp = tc::smem_desc(grp_addr + L::kP, 128, 1024, tc::kSwizzleNone);
            for (int n = g; n < cnt; n += kStGroups) {
                const int islot = n % kStInfoSlots;
                const uint32_t iph = (uint32_t)(n / kStInfoSlots) & 1u;
                const uint32_t mph = (uint32_t)(n / kStGroups) & 1u;
                wait(bar_info_full(islot), iph);
                const int *meta = reinterpret_cast<const int *>(smem + L::kInfo0 + islot * L::kInfoBytes + L::kMeta);
                const int n_tok = meta[3], tile0 = meta[4];
                tc::mbar_arrive(bar_info_empty(islot));
                const int n_tiles = n_tok > kStTile ? 2 : 1;
                int st[4];       // stages of K tile 0, K tile 1, V tile 0, V tile 1 (the chunk's tiles in ring order)
                uint32_t ph[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const unsigned gi = (unsigned)(tile0 + i);   // (unsigned: after a wait that ran out the record may hold anything, and the stage index must stay inside the ring)
                    st[i] = (int)(gi % (unsigned)S);
                    ph[i] = (gi / (unsigned)S) & 1u;
                }
                // ---- scores: S^T[token][head] = K_codes . Q^T; each K stage goes back to the producer when read
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    if (t < n_tiles) wait(bar_full(st[t]), ph[t]);
                wait(bar_ready_s(g), mph);
                tc::fence_after_sync();
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (t < n_tiles) {
                        const uint64_t a = dk0 + (uint64_t)((uint32_t)st[t] * (kStTileBytes >> 4));
#pragma unroll
                        for (int j = 0; j < 4; ++j)   // 32 dims per step: 32 bytes inside the swizzle span; 256 bytes of the query operand
                            tc::mma_i8(tm + t * NS, a + (uint64_t)(j * 2), dq + (uint64_t)(j * 16), idesc_s, j > 0);
                    }
                }
                tc::commit(bar_mma_s(g));
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    if (t < n_tiles) tc::commit(bar_empty(st[t]));
                // ---- output: O^T[dim][head] = V_codes^T . P^T
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    if (t < n_tiles) wait(bar_full(st[n_tiles + t]), ph[n_tiles + t]);
                wait(bar_ready_pv(g), mph);
                tc::fence_after_sync();
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (t < n_tiles) {
                        const uint64_t a = dv0 + (uint64_t)((uint32_t)st[n_tiles + t] * (kStTileBytes >> 4));
#pragma unroll
                        for (int j = 0; j < 4; ++j)   // 32 tokens per step: 4 KB down the V tile; 256 bytes of the P^T tile
                            tc::mma_i8(tm + 2 * NS, a + (uint64_t)(j * 256), dp + (uint64_t)((t * L::kPTileBytes + j * 256) >> 4), idesc_pv,
                                       (t > 0) || (j > 0));
                    }
                }
                tc::commit(bar_mma_pv(g));
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    if (t < n_tiles) tc::commit(bar_empty(st[n_tiles + t]));
            }
        }
    } else {
        // =========================================================== consumers: thread = token (tile 0: gtid, tile 1: 128 + gtid)
        const int g = warp >> 2, gtid = tid & 127, gw = warp & 3;
        unsigned char *grp = smem + L::kGroup0 + g * L::kGroupBytes;
        float *lsum = reinterpret_cast<float *>(grp + L::kLsum);   // [NH][128]
        float *red_m = reinterpret_cast<float *>(grp + L::kRed);   // [NH][4]
        float *rowscale = red_m + 4 * NH;                          // [NH]
        const uint32_t tm = tmem + (uint32_t)g * 128u;             // this group's columns: S tile 0 | S tile 1 | O
        const uint32_t lane_base = (uint32_t)(gw * 32) << 16;
        const int bar_id = 1 + g;
        int q_b = -1, q_head = -1;                                 // whose query rows the operand buffer holds

        {
            // ---- the last token of every (sequence, kv head) is attended from registers, here, while the first tiles
            //      are on their way (st_last_token).  A pair with chunks belongs to the block whose range holds its
            //      last chunk; those pairs are dealt to the block's consumer warps in turn, from the last warp down (the
            //      first group takes the block's first chunk).  A sequence of one token has no chunk: its pairs are
            //      dealt to the blocks by index.
            pdl_wait();
            if (cnt > 0) {
                int b = range[1], head = range[2];
                int L = range[5] + 1;   // the chunks cover all of the sequence's tokens but the last
                int nc = range[4];
                int last = nc - 1 - range[3];   // list index of the pair's last chunk
                for (int r = 0; last < cnt; ++r) {
                    if (kPW - 1 - r % kPW == warp) st_last_token<kAppend>(p, b, head, L, nc, lane, false);
                    // the next pair with chunks
                    if (++head == p.Hkv) {
                        head = 0;
                        do {
                            ++b;
                            L = (b < B) ? st_clamped_len(p, b) : 0;
                        } while (b < B && L < 2);
                        if (b >= B) break;
                        nc = (L - 1 + kStChunk - 1) / kStChunk;
                    }
                    last += nc;
                }
            }
            const long long pairs = (long long)B * p.Hkv;
            for (long long pr = blockIdx.x + (long long)warp * gridDim.x; pr < pairs; pr += (long long)kPW * gridDim.x) {
                const int b = (int)st_div(pr, p.Hkv), head = (int)(pr - (long long)b * p.Hkv);
                if (st_clamped_len(p, b) == 1) st_last_token<kAppend>(p, b, head, 1, 0, lane, kMerge);
            }
        }
        for (int n = g; n < cnt; n += kStGroups) {
            const int islot = n % kStInfoSlots;
            const uint32_t iph = (uint32_t)(n / kStInfoSlots) & 1u;
            const uint32_t mph = (uint32_t)(n / kStGroups) & 1u;
            const unsigned char *info = smem + L::kInfo0 + islot * L::kInfoBytes;
            wait(bar_info_full(islot), iph);
            const int *meta = reinterpret_cast<const int *>(info + L::kMeta);
            const int b = meta[0], head = meta[1], chunk = meta[2], n_tok = meta[3];
            const bool record_ok = ok;   // false: the wait for the record ran out and its fields may hold anything - nothing is written to global memory from them
            const int n_tiles = n_tok > kStTile ? 2 : 1;
            const int h0 = head * p.G;

            // ---- query operand (only when the chunk belongs to another (sequence, kv head) than the last one):
            //      warp w converts heads w, w+4, ...; a lane owns four consecutive dims
            if (b != q_b || head != q_head) {
                q_b = b;
                q_head = head;
                for (int h = gw; h < p.G; h += 4) {
                    const uint2 raw = *reinterpret_cast<const uint2 *>(info + L::kQraw + h * 256 + lane * 8);
                    const float x[4] = {bf16_bits_to_float(raw.x & 0xFFFFu), bf16_bits_to_float(raw.x >> 16),
                                        bf16_bits_to_float(raw.y & 0xFFFFu), bf16_bits_to_float(raw.y >> 16)};
                    const float am = warp_max(fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3]))));
                    const float p2 = pow2_floor(am);
                    const float f = pow2_recip(p2) * kStQFix;
                    uint32_t lo_w = 0, mid_w = 0, hi_w = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        // v = round(x * f), |v| < 2^21, as v = 65536 hi + 256 mid + lo with mid, lo in [-128, 127]
                        const int v = __float2int_rn(x[i] * f);
                        const int lo = (v << 24) >> 24;
                        const int v1 = (v - lo) >> 8;
                        const int mid = (v1 << 24) >> 24;
                        const int hi = (v1 - mid) >> 8;
                        lo_w |= ((uint32_t)lo & 0xFFu) << (8 * i);
                        mid_w |= ((uint32_t)mid & 0xFFu) << (8 * i);
                        hi_w |= ((uint32_t)hi & 0xFFu) << (8 * i);
                    }
                    if (lane == 0) rowscale[h] = p2 * p.scale_log2e * (1.f / kStQFix);
                    *reinterpret_cast<uint32_t *>(grp + L::kQop + st_core_off(h, 4 * lane)) = hi_w;
                    *reinterpret_cast<uint32_t *>(grp + L::kQop + st_core_off(NH + h, 4 * lane)) = mid_w;
                    *reinterpret_cast<uint32_t *>(grp + L::kQop + st_core_off(2 * NH + h, 4 * lane)) = lo_w;
                }
            }
            // this thread's two tokens
            float sk[2], lsv[2], rsv[2];
            bool valid[2];
            {
                const float *sc = reinterpret_cast<const float *>(info + L::kScales);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int tok = t * kStTile + gtid;
                    valid[t] = tok < n_tok;
                    const float sv = valid[t] ? fmaxf(sc[t * 256 + 128 + gtid], kMinScale) : 1.f;
                    sk[t] = valid[t] ? sc[t * 256 + gtid] : 0.f;
                    lsv[t] = __log2f(sv);
                    rsv[t] = valid[t] ? st_rcp(sv) : 0.f;
                }
            }
            tc::mbar_arrive(bar_info_empty(islot));   // this thread has read everything it needs from the record
            tc::fence_proxy_async();
            tc::mbar_arrive(bar_ready_s(g));          // the query operand is in place (128 arrivals start the score MMAs)

            wait(bar_mma_s(g), mph);
            __syncwarp();   // reconverge after the wait loop: the tensor-memory loads below are warp-aligned
            tc::fence_after_sync();

            // ---- S^T from tensor memory: row = token, columns [hi | mid | lo] per head
            float s[2][NH];
            float mloc[NH];
#pragma unroll
            for (int h = 0; h < NH; ++h) mloc[h] = -INFINITY;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (t < n_tiles) {
                    uint32_t r[NS];
#pragma unroll
                    for (int c16 = 0; c16 < NS / 16; ++c16) {
                        uint32_t tmp[16];
                        tc::tmem_ld16(tm + lane_base + t * NS + c16 * 16, tmp);
#pragma unroll
                        for (int i = 0; i < 16; ++i) r[c16 * 16 + i] = tmp[i];
                    }
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int h = 0; h < NH; ++h) {
                        // 65536 hi + 256 mid + lo; each plane's sum is below 2^22 in magnitude
                        const float x = fmaf((float)(int)r[h], 65536.f, (float)(((int)r[NH + h] << 8) + (int)r[2 * NH + h]));
                        s[t][h] = (valid[t] && h < p.G) ? fmaf(x, sk[t] * rowscale[h], lsv[t]) : -INFINITY;
                        mloc[h] = fmaxf(mloc[h], s[t][h]);
                    }
                } else {
#pragma unroll
                    for (int h = 0; h < NH; ++h) s[t][h] = -INFINITY;
                }
            }
            // warp maxima by one integer reduction per head (the map float -> int below preserves the order)
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                if (h < p.G) {
                    const int m = __reduce_max_sync(0xffffffffu, st_ordered_int(mloc[h]));
                    if (lane == 0) red_m[h * 4 + gw] = st_ordered_float(m);
                }
            }
            tc::fence_before_sync();
            tc::named_barrier(bar_id, kStGroupThreads);

            // ---- one softmax over the chunk's scores per head; P^T as bytes [hi | lo]
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                if (h < p.G) {
                    const float4 mw = *reinterpret_cast<const float4 *>(red_m + h * 4);
                    const float M = fmaxf(fmaxf(mw.x, mw.y), fmaxf(mw.z, mw.w));
                    float lloc = 0.f;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (t < n_tiles) {
                            const float e = st_exp2(s[t][h] - M);
                            lloc = fmaf(e, rsv[t], lloc);
                            const uint32_t bits = __float_as_uint(fmaf(e, kStPFix, 8388608.f));   // 2^23 + round(e * 65535)
                            unsigned char *pt = grp + L::kP + t * L::kPTileBytes;
                            pt[st_core_off(h, gtid)] = (unsigned char)((bits >> 8) & 0xFFu);
                            pt[st_core_off(NH + h, gtid)] = (unsigned char)(bits & 0xFFu);
                        }
                    }
                    lsum[h * kStGroupThreads + gtid] = lloc;
                }
            }
            tc::fence_proxy_async();
            tc::mbar_arrive(bar_ready_pv(g));         // P^T is in place (128 arrivals start the output MMAs)

            wait(bar_mma_pv(g), mph);
            __syncwarp();
            tc::fence_after_sync();

            // ---- O^T from tensor memory: row = head dim, columns [hi | lo] per head; one partial per head
            {
                uint32_t r[NP];
#pragma unroll
                for (int c16 = 0; c16 < NP / 16; ++c16) {
                    uint32_t tmp[16];
                    tc::tmem_ld16(tm + lane_base + 2 * NS + c16 * 16, tmp);
#pragma unroll
                    for (int i = 0; i < 16; ++i) r[c16 * 16 + i] = tmp[i];
                }
                tc::tmem_ld_wait();
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    if (h < p.G && record_ok) {
                        const size_t ps = ((size_t)b * p.Hq + h0 + h) * p.n_slots + chunk;
                        p.part_o[ps * kHeadDim + gtid] = (float)(((int)r[h] << 8) + (int)r[NH + h]) * (1.f / kStPFix);
                    }
                }
            }
            // ---- denominators: 128 / NH consecutive lanes add up one head's 128 shares (all of them were written
            //      before the output MMAs started)
            {
                constexpr int kLanesPerHead = kStGroupThreads / NH;   // 16 or 8
                const int h = gtid / kLanesPerHead, seg = gtid % kLanesPerHead;
                const float4 *src = reinterpret_cast<const float4 *>(lsum + h * kStGroupThreads + seg * NH);
                float l = 0.f;
#pragma unroll
                for (int i = 0; i < NH / 4; ++i) {
                    const float4 v = src[i];
                    l += (v.x + v.y) + (v.z + v.w);
                }
#pragma unroll
                for (int o = kLanesPerHead / 2; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
                if (seg == 0 && h < p.G && record_ok) {
                    const size_t ps = ((size_t)b * p.Hq + h0 + h) * p.n_slots + chunk;
                    const float4 mw = *reinterpret_cast<const float4 *>(red_m + h * 4);
                    p.part_ml[ps * 2] = fmaxf(fmaxf(mw.x, mw.y), fmaxf(mw.z, mw.w));
                    p.part_ml[ps * 2 + 1] = l;
                }
            }
            // the next chunk's MMAs overwrite this group's tensor-memory columns: the loads above have retired
            tc::fence_before_sync();
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    if (kMerge) {
        // ---- the block's partials are written: merge what is complete.  A (sequence, kv head) whose chunks all lie
        //      in this block's range is merged at once; one that is shared with other blocks is counted in global
        //      memory (every block adds its number of chunks) and merged by the block whose count completes it.
        __threadfence();   // this thread's partials are visible device-wide before any count that includes them
        __syncthreads();
        if (warp < kPW) {
            if (cnt > 0) {
                int b = range[1], head = range[2], first = range[3], nc = range[4];
                int remaining = cnt;
                for (int r = 0; remaining > 0; ++r) {
                    const int mine = min(nc - first, remaining);
                    if (r % kPW == warp) {
                        // the block that holds the pair's last chunk also wrote the last token's partial (slot nc)
                        const int wrote = mine + ((first + mine == nc) ? 1 : 0);
                        bool complete = mine == nc;
                        if (!complete) {
                            int old = 0;
                            if (lane == 0) old = atomicAdd(p.counters + b * p.Hkv + head, wrote);
                            complete = __shfl_sync(0xffffffffu, old, 0) + wrote == nc + 1;
                            if (complete) {
                                if (lane == 0) p.counters[b * p.Hkv + head] = 0;   // ready for the next launch
                                __threadfence();   // the other blocks' counts were seen: their partials are visible after this
                            }
                        }
                        if (complete) st_merge_rows(p, b, head, nc + 1, lane);
                    }
                    remaining -= mine;
                    first = 0;
                    if (remaining > 0 && ++head == p.Hkv) {
                        head = 0;
                        int len;
                        do {
                            ++b;
                            len = (b < B) ? st_chunk_len(p, b) : kStChunk;   // b < B always holds inside the range
                        } while (len == 0);
                        nc = (len + kStChunk - 1) / kStChunk;
                    }
                }
            }
            // sequences without tokens have no partial and therefore no merge: their rows are zero (a sequence of one
            // token was written by the warp that attended it)
            for (int b = blockIdx.x; b < B; b += gridDim.x) {
                if (st_clamped_len(p, b) != 0) continue;
                uint4 *dst = reinterpret_cast<uint4 *>(p.out + (size_t)b * p.Hq * kHeadDim);
                for (int i = tid; i < p.Hq * (kHeadDim / 8); i += kPW * 32) dst[i] = make_uint4(0, 0, 0, 0);
            }
        }
    }
    if (warp == kPW) {
        if (lane == 0 && *fail != 0) {
            // a wait ran out somewhere: give the copies still in flight a bounded chance to land before the block exits
            for (int gi = max(0, tiles_issued - S); gi < tiles_issued; ++gi)
                tc::mbar_wait(bar_full(gi % S), (uint32_t)(gi / S) & 1u, 1u << 14);
            for (int n = max(0, cnt - kStInfoSlots); n < cnt; ++n)
                tc::mbar_wait(bar_info_full(n % kStInfoSlots), (uint32_t)(n / kStInfoSlots) & 1u, 1u << 14);
            if (p.status != nullptr) atomicExch(p.status, SLIM_ERR_TIMEOUT);
        }
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(*tmem_slot, L::kTmemCols);   // (this warp allocated it; the block's last barrier lies behind)
    }
}

template <int NH, bool kAppend, bool kMerge>
static int launch_stream(dim3 grid, cudaStream_t stream, const CUtensorMap &map_tile, const CUtensorMap &map_tail,
                         const DecodeParams &p, int B)
{
    constexpr int bytes = (int)StSmem<NH, kAppend>::kBytes;
    const int rc = allow_dynamic_smem(reinterpret_cast<const void *>(slim_decode_stream_kernel<NH, kAppend, kMerge>), bytes);
    if (rc != SLIM_OK) return rc;
    SLIM_CUDA_TRY(launch_pdl(slim_decode_stream_kernel<NH, kAppend, kMerge>, grid, dim3(StSmem<NH, kAppend>::kThreads), bytes, stream, map_tile,
                             map_tail, p, B));
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

int launch_decode_split_stream(const slim_cache_t *c, const DecodeParams &p, int B, cudaStream_t stream)
{
    CUtensorMap map_tile, map_tail;
    int rc = codes_tensor_map(c, kStTile, &map_tile);
    if (rc != SLIM_OK) return rc;
    rc = codes_tensor_map(c, kStTailBox, &map_tail);
    if (rc != SLIM_OK) return rc;
    int sms = 0;
    rc = sm_count(&sms);
    if (rc != SLIM_OK) return rc;
    const long long max_items = (long long)p.n_chunks * p.Hkv * B;
    const unsigned grid = (unsigned)(max_items < sms ? max_items : sms);
    const dim3 blocks(grid);
    const bool append = p.k_new != nullptr, merge = p.counters != nullptr;
    if (p.G <= 8) {
        if (merge) {
            if (append) return launch_stream<8, true, true>(blocks, stream, map_tile, map_tail, p, B);
            return launch_stream<8, false, true>(blocks, stream, map_tile, map_tail, p, B);
        }
        if (append) return launch_stream<8, true, false>(blocks, stream, map_tile, map_tail, p, B);
        return launch_stream<8, false, false>(blocks, stream, map_tile, map_tail, p, B);
    }
    if (merge) {
        if (append) return launch_stream<16, true, true>(blocks, stream, map_tile, map_tail, p, B);
        return launch_stream<16, false, true>(blocks, stream, map_tile, map_tail, p, B);
    }
    if (append) return launch_stream<16, true, false>(blocks, stream, map_tile, map_tail, p, B);
    return launch_stream<16, false, false>(blocks, stream, map_tile, map_tail, p, B);
}

}  // namespace slim

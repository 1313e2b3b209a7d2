// Parameters shared by the decode split kernels and the merge kernel.
#pragma once
#include "slim_common.cuh"

namespace slim {

struct DecodeParams {
    const int8_t *codes;
    const float *scales;
    const int32_t *block_table;
    const int32_t *kv_len;
    const __nv_bfloat16 *q;   // [B][Hq][128]
    int *status;              // first word of the workspace: set to a SLIM_ERR_* code by a kernel whose wait ran out
    float *part_o;            // [B][Hq][n_slots][128] unnormalised partial outputs: a row's chunks, then its last token
    float *part_ml;           // [B][Hq][n_slots][2]   (max in log2 units, sum)
    // one-kernel append + split (optional): the new token of every sequence, [B][Hkv][128], quantised into slot
    // kv_len - 1 by the warp that attends the sequence's last token (null: nothing to append)
    const __nv_bfloat16 *k_new, *v_new;
    // merge at the end of the split kernel (optional, both or neither): the result [B][Hq][128] and the counters
    // [B * Hkv] of chunks counted so far per (sequence, kv head); zero before and after every launch
    __nv_bfloat16 *out;
    int *counters;
    int Hq, Hkv, G;
    int max_pages_per_seq, num_pages;
    int n_chunks;             // 256-token chunks that max_kv tokens need
    int n_slots;              // partial slots per row: n_chunks + 1 (the last token of a row has a partial of its own)
    float scale_log2e;        // sm_scale * log2(e)
};

// Workspace header in front of the partials: the status word (16 bytes), then the counters of the in-kernel
// merge.  The header has one size for every shape, so a workspace zeroed once stays valid when the shapes of the
// calls that use it change.
constexpr size_t kDecodeStatusBytes = 16;
constexpr int kDecodeCounterRows = 16384;   // (sequence, kv head) pairs the in-kernel merge can count
constexpr size_t kDecodeHeaderBytes = kDecodeStatusBytes + (size_t)kDecodeCounterRows * sizeof(int);

int launch_decode_split_stream(const slim_cache_t *c, const DecodeParams &p, int B, cudaStream_t stream);

}  // namespace slim

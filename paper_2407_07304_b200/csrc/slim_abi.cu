// C ABI of the library (declared in include/slim.h): argument validation and dispatch.
#include "slim_common.cuh"
#include "slim_tcgen05.cuh"

#define SLIM_EXPORT extern "C" __attribute__((visibility("default")))

namespace slim {

static thread_local int g_last_cuda_error = 0;

int set_cuda_error(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    return SLIM_ERR_CUDA;
}

int launch_append(const slim_cache_t *c, const void *k_new, const void *v_new, const int32_t *cu_new,
                  const int32_t *start_pos, int B, int max_new, cudaStream_t stream, const int32_t *len_after);
int launch_decode_split(const slim_cache_t *c, const void *q, const void *k_new, const void *v_new, const int32_t *kv_len,
                        int B, int max_kv, int Hq, float sm_scale, void *workspace, cudaStream_t stream);
int launch_decode_merge(const slim_cache_t *c, void *out, const int32_t *kv_len, int B, int max_kv, int Hq,
                        const void *workspace, cudaStream_t stream, float *raw = nullptr);
int launch_decode(const slim_cache_t *c, const void *q, const void *k_new, const void *v_new, void *out,
                  const int32_t *kv_len, int B, int max_kv, int Hq, float sm_scale, void *workspace, cudaStream_t stream);
int launch_decode_partial(const slim_cache_t *c, const void *q, float *partial, const int32_t *kv_len, int B, int max_kv, int Hq,
                          float sm_scale, void *workspace, cudaStream_t stream);
int launch_merge_partials(const float *parts, int R, int rows, void *out, cudaStream_t stream);
size_t decode_workspace_bytes(int B, int Hq, int Hkv, int max_kv);
int launch_prefill_tc(const slim_cache_t *c, const void *q, void *out, const int32_t *cu_q, const int32_t *kv_len,
                      int B, int max_q, int Hq, float sm_scale, void *workspace, cudaStream_t stream, bool two_pass, bool after_append);
int launch_prefill_row(const slim_cache_t *c, const void *q, void *out, const int32_t *cu_q, const int32_t *kv_len,
                       int B, int max_q, int Hq, float sm_scale, void *workspace, cudaStream_t stream);
size_t prefill_workspace_bytes();

static int check_cache(const slim_cache_t *c)
{
    if (c == nullptr || c->codes == nullptr || c->scales == nullptr || c->block_table == nullptr)
        return SLIM_ERR_INVALID_ARG;
    if (c->num_pages <= 0 || c->num_kv_heads <= 0 || c->max_pages_per_seq <= 0) return SLIM_ERR_INVALID_ARG;
    if (c->page_tokens != SLIM_PAGE_TOKENS || c->head_dim != SLIM_HEAD_DIM) return SLIM_ERR_UNSUPPORTED;
    if (((uintptr_t)c->codes & 15) || ((uintptr_t)c->scales & 15)) return SLIM_ERR_INVALID_ARG;
    return SLIM_OK;
}

}  // namespace slim

using namespace slim;

SLIM_EXPORT int slim_kv_append(const slim_cache_t *cache, const void *k_new, const void *v_new,
                               const int32_t *cu_new, const int32_t *start_pos, int32_t B, int32_t max_new,
                               void *stream)
{
    int rc = check_cache(cache);
    if (rc != SLIM_OK) return rc;
    if (B < 0 || max_new < 0) return SLIM_ERR_INVALID_ARG;
    if (B == 0 || max_new == 0) return SLIM_OK;
    if (k_new == nullptr || v_new == nullptr || cu_new == nullptr || start_pos == nullptr) return SLIM_ERR_INVALID_ARG;
    if (((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15)) return SLIM_ERR_INVALID_ARG;   // rows are read 16 bytes at a time
    if (B > 65535) return SLIM_ERR_UNSUPPORTED;
    return launch_append(cache, k_new, v_new, cu_new, start_pos, B, max_new, (cudaStream_t)stream, nullptr);
}

enum PrefillVariant { kPrefillStreamed, kPrefillTwoPass, kPrefillFullRow };

// Shared validation of the prefill entry points; *launch is false for a valid no-op.
static int check_prefill(const slim_cache_t *cache, const void *q, const void *out, const int32_t *cu_q, const int32_t *kv_len,
                         int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq, const void *workspace, size_t workspace_bytes,
                         bool *launch)
{
    *launch = false;
    int rc = check_cache(cache);
    if (rc != SLIM_OK) return rc;
    if (B < 0 || max_q < 0 || max_kv < 0 || Hq <= 0) return SLIM_ERR_INVALID_ARG;
    if (Hq % cache->num_kv_heads != 0) return SLIM_ERR_UNSUPPORTED;
    if (B == 0 || max_q == 0) return SLIM_OK;
    if (q == nullptr || out == nullptr || cu_q == nullptr || kv_len == nullptr) return SLIM_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return SLIM_ERR_INVALID_ARG;
    if (B > 65535 || Hq > 65535) return SLIM_ERR_UNSUPPORTED;
    if ((long long)max_kv > (long long)cache->max_pages_per_seq * SLIM_PAGE_TOKENS) return SLIM_ERR_INVALID_ARG;
    const size_t need = slim_workspace_bytes(SLIM_PHASE_PREFILL, B, Hq, cache->num_kv_heads, max_q, max_kv);
    if (need > 0 && (workspace == nullptr || workspace_bytes < need)) return SLIM_ERR_WORKSPACE;
    *launch = true;
    return SLIM_OK;
}

static int prefill_entry(const slim_cache_t *cache, const void *q, void *out, const int32_t *cu_q,
                         const int32_t *kv_len, int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq,
                         float sm_scale, void *workspace, size_t workspace_bytes, void *stream, PrefillVariant variant)
{
    bool launch;
    const int rc = check_prefill(cache, q, out, cu_q, kv_len, B, max_q, max_kv, Hq, workspace, workspace_bytes, &launch);
    if (rc != SLIM_OK || !launch) return rc;
    if (variant == kPrefillFullRow) {
        if (max_kv > SLIM_FULL_ROW_MAX_KEYS) return SLIM_ERR_UNSUPPORTED;   // the score strip of a row block must fit tensor memory
        return launch_prefill_row(cache, q, out, cu_q, kv_len, B, max_q, Hq, sm_scale, workspace, (cudaStream_t)stream);
    }
    return launch_prefill_tc(cache, q, out, cu_q, kv_len, B, max_q, Hq, sm_scale, workspace, (cudaStream_t)stream,
                             variant == kPrefillTwoPass, false);
}

// The first-token phase in one call: the prompt's K / V rows are quantised into the cache and the attention over
// the cache follows, the second kernel launched so that its set-up and its query rows overlap the end of the first.
SLIM_EXPORT int slim_prefill_step(const slim_cache_t *cache, const void *q, const void *k_new, const void *v_new, void *out,
                                  const int32_t *cu_q, const int32_t *kv_len, int32_t B, int32_t max_q, int32_t max_kv,
                                  int32_t Hq, float sm_scale, void *workspace, size_t workspace_bytes, void *stream)
{
    bool launch;
    int rc = check_prefill(cache, q, out, cu_q, kv_len, B, max_q, max_kv, Hq, workspace, workspace_bytes, &launch);
    if (rc != SLIM_OK || !launch) return rc;
    if (k_new == nullptr || v_new == nullptr || ((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15)) return SLIM_ERR_INVALID_ARG;
    // the new rows of sequence b go to positions kv_len[b] - q_len[b] ... kv_len[b] - 1
    rc = launch_append(cache, k_new, v_new, cu_q, nullptr, B, max_q, (cudaStream_t)stream, kv_len);
    if (rc != SLIM_OK) return rc;
    return launch_prefill_tc(cache, q, out, cu_q, kv_len, B, max_q, Hq, sm_scale, workspace, (cudaStream_t)stream, false, true);
}

SLIM_EXPORT int slim_attn_prefill(const slim_cache_t *cache, const void *q, void *out, const int32_t *cu_q,
                                  const int32_t *kv_len, int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq,
                                  float sm_scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return prefill_entry(cache, q, out, cu_q, kv_len, B, max_q, max_kv, Hq, sm_scale, workspace, workspace_bytes, stream, kPrefillStreamed);
}

SLIM_EXPORT int slim_attn_prefill_two_pass(const slim_cache_t *cache, const void *q, void *out, const int32_t *cu_q,
                                           const int32_t *kv_len, int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq,
                                           float sm_scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return prefill_entry(cache, q, out, cu_q, kv_len, B, max_q, max_kv, Hq, sm_scale, workspace, workspace_bytes, stream, kPrefillTwoPass);
}

SLIM_EXPORT int slim_attn_prefill_full_row(const slim_cache_t *cache, const void *q, void *out, const int32_t *cu_q,
                                           const int32_t *kv_len, int32_t B, int32_t max_q, int32_t max_kv, int32_t Hq,
                                           float sm_scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return prefill_entry(cache, q, out, cu_q, kv_len, B, max_q, max_kv, Hq, sm_scale, workspace, workspace_bytes, stream, kPrefillFullRow);
}

// Shared validation of the decode entry points; *launch is false for a valid no-op.
static int check_decode(const slim_cache_t *cache, int32_t B, int32_t max_kv, int32_t Hq, const void *workspace,
                        size_t workspace_bytes, bool *launch)
{
    *launch = false;
    int rc = check_cache(cache);
    if (rc != SLIM_OK) return rc;
    if (B < 0 || max_kv < 0 || Hq <= 0) return SLIM_ERR_INVALID_ARG;
    if (Hq % cache->num_kv_heads != 0 || Hq / cache->num_kv_heads > 16) return SLIM_ERR_UNSUPPORTED;
    if (B == 0) return SLIM_OK;
    if (B > 65535 || cache->num_kv_heads > 65535) return SLIM_ERR_UNSUPPORTED;
    if ((long long)max_kv > (long long)cache->max_pages_per_seq * SLIM_PAGE_TOKENS) return SLIM_ERR_INVALID_ARG;
    const size_t need = slim_workspace_bytes(SLIM_PHASE_DECODE, B, Hq, cache->num_kv_heads, 1, max_kv);
    if (need > 0 && (workspace == nullptr || workspace_bytes < need)) return SLIM_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 15) return SLIM_ERR_INVALID_ARG;
    *launch = true;
    return SLIM_OK;
}

SLIM_EXPORT int slim_attn_decode_split(const slim_cache_t *cache, const void *q, const void *k_new, const void *v_new,
                                       const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale,
                                       void *workspace, size_t workspace_bytes, void *stream)
{
    bool launch;
    int rc = check_decode(cache, B, max_kv, Hq, workspace, workspace_bytes, &launch);
    if (rc != SLIM_OK || !launch) return rc;
    if (q == nullptr || kv_len == nullptr || ((uintptr_t)q & 15)) return SLIM_ERR_INVALID_ARG;
    if ((k_new == nullptr) != (v_new == nullptr) || ((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15)) return SLIM_ERR_INVALID_ARG;
    return launch_decode_split(cache, q, k_new, v_new, kv_len, B, max_kv, Hq, sm_scale, workspace, (cudaStream_t)stream);
}

SLIM_EXPORT int slim_attn_decode_merge(const slim_cache_t *cache, void *out, const int32_t *kv_len, int32_t B,
                                       int32_t max_kv, int32_t Hq, const void *workspace, size_t workspace_bytes,
                                       void *stream)
{
    bool launch;
    int rc = check_decode(cache, B, max_kv, Hq, workspace, workspace_bytes, &launch);
    if (rc != SLIM_OK || !launch) return rc;
    if (out == nullptr || kv_len == nullptr || ((uintptr_t)out & 15)) return SLIM_ERR_INVALID_ARG;
    return launch_decode_merge(cache, out, kv_len, B, max_kv, Hq, workspace, (cudaStream_t)stream);
}

SLIM_EXPORT int slim_attn_decode(const slim_cache_t *cache, const void *q, void *out, const int32_t *kv_len,
                                 int32_t B, int32_t max_kv, int32_t Hq, float sm_scale, void *workspace,
                                 size_t workspace_bytes, void *stream)
{
    bool launch;
    int rc = check_decode(cache, B, max_kv, Hq, workspace, workspace_bytes, &launch);
    if (rc != SLIM_OK || !launch) return rc;
    if (q == nullptr || out == nullptr || kv_len == nullptr) return SLIM_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return SLIM_ERR_INVALID_ARG;
    return launch_decode(cache, q, nullptr, nullptr, out, kv_len, B, max_kv, Hq, sm_scale, workspace, (cudaStream_t)stream);
}

SLIM_EXPORT int slim_attn_decode_partial(const slim_cache_t *cache, const void *q, float *partial, const int32_t *kv_len,
                                         int32_t B, int32_t max_kv, int32_t Hq, float sm_scale, void *workspace,
                                         size_t workspace_bytes, void *stream)
{
    bool launch;
    int rc = check_decode(cache, B, max_kv, Hq, workspace, workspace_bytes, &launch);
    if (rc != SLIM_OK || !launch) return rc;
    if (q == nullptr || partial == nullptr || kv_len == nullptr) return SLIM_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)partial & 15)) return SLIM_ERR_INVALID_ARG;
    return launch_decode_partial(cache, q, partial, kv_len, B, max_kv, Hq, sm_scale, workspace, (cudaStream_t)stream);
}

SLIM_EXPORT int slim_attn_merge_partials(const float *partials, int32_t n_sets, void *out, int32_t B, int32_t Hq, void *stream)
{
    if (n_sets < 0 || B < 0 || Hq <= 0) return SLIM_ERR_INVALID_ARG;
    if (B == 0) return SLIM_OK;
    if (partials == nullptr || out == nullptr || n_sets == 0) return SLIM_ERR_INVALID_ARG;
    if (((uintptr_t)partials & 15) || ((uintptr_t)out & 15)) return SLIM_ERR_INVALID_ARG;
    if ((long long)B * Hq > 0x7FFFFFFFLL / SLIM_PARTIAL_FLOATS) return SLIM_ERR_UNSUPPORTED;
    return launch_merge_partials(partials, n_sets, B * Hq, out, (cudaStream_t)stream);
}

SLIM_EXPORT int slim_decode_step(const slim_cache_t *cache, const void *q, const void *k_new, const void *v_new, void *out,
                                 const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale,
                                 void *workspace, size_t workspace_bytes, void *stream)
{
    bool launch;
    int rc = check_decode(cache, B, max_kv, Hq, workspace, workspace_bytes, &launch);
    if (rc != SLIM_OK || !launch) return rc;
    if (q == nullptr || k_new == nullptr || v_new == nullptr || out == nullptr || kv_len == nullptr) return SLIM_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15) || ((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15))
        return SLIM_ERR_INVALID_ARG;
    return launch_decode(cache, q, k_new, v_new, out, kv_len, B, max_kv, Hq, sm_scale, workspace, (cudaStream_t)stream);
}

SLIM_EXPORT size_t slim_step_staging_bytes(int32_t B, int32_t Hq, int32_t Hkv)
{
    if (B <= 0 || Hq <= 0 || Hkv <= 0) return 0;
    return ((size_t)2 * B * Hq + (size_t)2 * B * Hkv) * SLIM_HEAD_DIM * 2;
}

SLIM_EXPORT int slim_decode_step_host(const slim_cache_t *cache, const void *q_host, const void *k_new_host,
                                      const void *v_new_host, void *out_host, void *staging, size_t staging_bytes,
                                      const int32_t *kv_len, int32_t B, int32_t max_kv, int32_t Hq, float sm_scale, void *workspace,
                                      size_t workspace_bytes, void *stream)
{
    bool launch;
    int rc = check_decode(cache, B, max_kv, Hq, workspace, workspace_bytes, &launch);
    if (rc != SLIM_OK || !launch) return rc;
    if (q_host == nullptr || k_new_host == nullptr || v_new_host == nullptr || out_host == nullptr || kv_len == nullptr)
        return SLIM_ERR_INVALID_ARG;
    const int Hkv = cache->num_kv_heads;
    if (staging == nullptr || ((uintptr_t)staging & 15) || staging_bytes < slim_step_staging_bytes(B, Hq, Hkv))
        return SLIM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t q_bytes = (size_t)B * Hq * SLIM_HEAD_DIM * 2, kv_bytes = (size_t)B * Hkv * SLIM_HEAD_DIM * 2;
    char *d_q = static_cast<char *>(staging), *d_k = d_q + q_bytes, *d_v = d_k + kv_bytes, *d_o = d_v + kv_bytes;
    const char *hq = static_cast<const char *>(q_host), *hk = static_cast<const char *>(k_new_host),
               *hv = static_cast<const char *>(v_new_host);
    // A pinned host buffer is mapped into the device's address space.  The kernel reads such inputs where they
    // are (every row is read once, by one warp or one bulk copy: the step moves the same bytes over the bus as a
    // copy would, without waiting for the copy first) and writes the result straight into such an output (visible
    // to the host once the stream has been synchronised).  Ordinary host memory goes through the staging buffer.
    auto mapped = [](const void *host) -> void * {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, host) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
            attr.devicePointer != nullptr && ((uintptr_t)attr.devicePointer & 15) == 0)
            return attr.devicePointer;
        (void)cudaGetLastError();   // an unregistered host pointer is not an error here: it takes the copy
        return nullptr;
    };
    const void *in_q = mapped(hq), *in_k = mapped(hk), *in_v = mapped(hv);
    if (in_q == nullptr || in_k == nullptr || in_v == nullptr) {
        if (hk == hq + q_bytes && hv == hk + kv_bytes) {
            // the three host buffers are adjacent (one allocation): one copy instead of three
            SLIM_CUDA_TRY(cudaMemcpyAsync(d_q, hq, q_bytes + 2 * kv_bytes, cudaMemcpyHostToDevice, st));
        } else {
            SLIM_CUDA_TRY(cudaMemcpyAsync(d_q, hq, q_bytes, cudaMemcpyHostToDevice, st));
            SLIM_CUDA_TRY(cudaMemcpyAsync(d_k, hk, kv_bytes, cudaMemcpyHostToDevice, st));
            SLIM_CUDA_TRY(cudaMemcpyAsync(d_v, hv, kv_bytes, cudaMemcpyHostToDevice, st));
        }
        in_q = d_q, in_k = d_k, in_v = d_v;
    }
    void *d_out = mapped(out_host);
    if (d_out == nullptr) d_out = d_o;
    rc = launch_decode(cache, in_q, in_k, in_v, d_out, kv_len, B, max_kv, Hq, sm_scale, workspace, st);
    if (rc != SLIM_OK) return rc;
    if (d_out == d_o) SLIM_CUDA_TRY(cudaMemcpyAsync(out_host, d_o, q_bytes, cudaMemcpyDeviceToHost, st));
    return SLIM_OK;
}

SLIM_EXPORT size_t slim_workspace_bytes(int32_t phase, int32_t B, int32_t Hq, int32_t Hkv, int32_t max_q,
                                        int32_t max_kv)
{
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || max_kv < 0 || max_q < 0) return 0;
    if (phase == SLIM_PHASE_DECODE) return decode_workspace_bytes(B, Hq, Hkv, max_kv);
    if (phase == SLIM_PHASE_PREFILL) return prefill_workspace_bytes();
    return 0;
}

SLIM_EXPORT int slim_read_status(const void *workspace, void *stream)
{
    if (workspace == nullptr) return SLIM_ERR_INVALID_ARG;
    int word = 0;
    SLIM_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    SLIM_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return (word == 0) ? SLIM_OK : SLIM_ERR_TIMEOUT;
}

// One thread waits on an mbarrier that nothing ever arrives on, with the same bounded wait the attention kernels
// use (a short limit here), and reports the way they do: SLIM_ERR_TIMEOUT in the status word, normal exit.
__global__ void slim_selftest_timeout_kernel(int *status)
{
    __shared__ __align__(8) unsigned long long mbar;
    const uint32_t addr = slim::smem_u32(&mbar);
    slim::tc::mbar_init(addr, 1);
    slim::tc::mbar_init_fence();
    if (!slim::tc::mbar_wait(addr, 0, 64u)) atomicExch(status, SLIM_ERR_TIMEOUT);
}

SLIM_EXPORT int slim_selftest_timeout(void *workspace, void *stream)
{
    if (workspace == nullptr || ((uintptr_t)workspace & 3)) return SLIM_ERR_INVALID_ARG;
    slim_selftest_timeout_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(static_cast<int *>(workspace));
    SLIM_CUDA_TRY(cudaGetLastError());
    return SLIM_OK;
}

SLIM_EXPORT size_t slim_cache_code_bytes(int32_t num_pages, int32_t num_kv_heads)
{
    if (num_pages <= 0 || num_kv_heads <= 0) return 0;
    return (size_t)num_pages * num_kv_heads * 2 * SLIM_PAGE_TOKENS * SLIM_HEAD_DIM;
}

SLIM_EXPORT size_t slim_cache_scale_bytes(int32_t num_pages, int32_t num_kv_heads)
{
    if (num_pages <= 0 || num_kv_heads <= 0) return 0;
    return (size_t)num_pages * num_kv_heads * 2 * SLIM_PAGE_TOKENS * sizeof(float);
}

SLIM_EXPORT const char *slim_strerror(int code)
{
    switch (code) {
        case SLIM_OK: return "ok";
        case SLIM_ERR_INVALID_ARG: return "invalid argument";
        case SLIM_ERR_UNSUPPORTED: return "unsupported shape";
        case SLIM_ERR_WORKSPACE: return "workspace missing or too small";
        case SLIM_ERR_CUDA: return "CUDA runtime error";
        case SLIM_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error";
    }
}

SLIM_EXPORT int slim_last_cuda_error(void) { return g_last_cuda_error; }

SLIM_EXPORT int slim_version(void) { return 100; }

// TMA tensor maps of the INT8 code pool (host side).
//
// The pool [num_pages][Hkv][2][128 slots][128 dims] is described to the copy engine as a 2-D
// byte tensor [rows][128] with rows = num_pages * Hkv * 2 * 128: one row per cached (token, kv
// head, K|V) vector.  A box of `box_rows` rows lands in shared memory with the 128-byte swizzle,
// which is the layout the tensor cores read directly.  x is always 0 (16-byte rule trivially met).
#include <cuda.h>

#include <mutex>

#include "slim_common.cuh"
#include "slim_tmap.cuh"

namespace slim {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct Entry {
    const void *ptr;
    long long rows;
    int box_rows;
    CUtensorMap map;
};
constexpr int kEntries = 32;
}  // namespace

int codes_tensor_map(const slim_cache_t *c, int box_rows, CUtensorMap *out)
{
    static std::mutex mu;
    static EncodeTiledFn encode = nullptr;
    static Entry cache[kEntries];
    static int used = 0, next = 0;
    std::lock_guard<std::mutex> lock(mu);
    if (encode == nullptr) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        SLIM_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return SLIM_ERR_UNSUPPORTED;
        encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    const long long rows = (long long)c->num_pages * c->num_kv_heads * 2 * kPageTokens;
    for (int i = 0; i < used; ++i) {
        if (cache[i].ptr == c->codes && cache[i].rows == rows && cache[i].box_rows == box_rows) {
            *out = cache[i].map;
            return SLIM_OK;
        }
    }
    Entry e;
    e.ptr = c->codes;
    e.rows = rows;
    e.box_rows = box_rows;
    const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kHeadDim};
    const cuuint32_t box[2] = {(cuuint32_t)kHeadDim, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(&e.map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(c->codes), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return SLIM_ERR_CUDA;
    cache[next] = e;
    next = (next + 1) % kEntries;
    if (used < kEntries) ++used;
    *out = e.map;
    return SLIM_OK;
}

int sm_count(int *out)
{
    static int cached[64];
    int dev = 0;
    SLIM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SLIM_ERR_UNSUPPORTED;
    if (cached[dev] == 0) {
        int n = 0;
        SLIM_CUDA_TRY(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
        cached[dev] = n;
    }
    *out = cached[dev];
    return SLIM_OK;
}

int allow_dynamic_smem(const void *func, int bytes)
{
    struct Done {
        int dev;
        const void *func;
    };
    static std::mutex mu;
    static Done done[64];
    static int n_done = 0;
    int dev = 0;
    SLIM_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_done; ++i)
        if (done[i].dev == dev && done[i].func == func) return SLIM_OK;
    SLIM_CUDA_TRY(cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    if (n_done < 64) done[n_done++] = Done{dev, func};
    return SLIM_OK;
}

}  // namespace slim

// Host-side TMA descriptor encoding.  The driver entry point is looked up through the runtime so
// that the library does not link against libcuda.
#include <mutex>

#include "tc05.cuh"

namespace swimba {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::once_flag g_once;

void lookup()
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
        g_encode = (EncodeTiledFn)fn;
    else
        cudaGetLastError();
}
}  // namespace

bool encode_tmap_bf16(CUtensorMap *out, const void *base, int rank, const uint64_t *dims,
                      const uint64_t *strides_bytes, const uint32_t *box)
{
    std::call_once(g_once, lookup);
    if (!g_encode || rank < 1 || rank > 5) return false;
    cuuint64_t gdim[5], gstr[4];
    cuuint32_t bdim[5], estr[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bdim[i] = box[i];
        estr[i] = 1;
        if (i + 1 < rank) gstr[i] = strides_bytes[i];
    }
    const CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
                                const_cast<void *>(base), gdim, gstr, bdim, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool encode_tmap_bf16_cached(TmapCache *cache, CUtensorMap *out, const void *base, int rank,
                             const uint64_t *dims, const uint64_t *strides_bytes, const uint32_t *box)
{
    if (!cache) return encode_tmap_bf16(out, base, rank, dims, strides_bytes, box);
    for (int i = 0; i < cache->used; ++i) {
        const TmapCache::Entry &c = cache->e[i];
        if (c.base != base || c.rank != rank) continue;
        bool same = true;
        for (int d = 0; d < rank && same; ++d) same = c.dims[d] == dims[d] && c.box[d] == box[d];
        for (int d = 0; d + 1 < rank && same; ++d) same = c.strides[d] == strides_bytes[d];
        if (same) {
            *out = c.map;
            return true;
        }
    }
    if (!encode_tmap_bf16(out, base, rank, dims, strides_bytes, box)) return false;
    TmapCache::Entry &c = cache->e[cache->next];
    c.base = base;
    c.rank = rank;
    for (int d = 0; d < rank; ++d) { c.dims[d] = dims[d]; c.box[d] = box[d]; }
    for (int d = 0; d + 1 < rank; ++d) c.strides[d] = strides_bytes[d];
    c.map = *out;
    cache->next = (cache->next + 1) % TmapCache::N;
    if (cache->used < TmapCache::N) cache->used++;
    return true;
}

namespace {
struct SmemAttr { const void *func; int device; size_t bytes; };
std::mutex g_attr_mutex;
SmemAttr g_attr[256];
int g_attr_n = 0;
}  // namespace

bool ensure_dynamic_smem(const void *func, size_t bytes)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(g_attr_mutex);
    SmemAttr *slot = nullptr;
    for (int i = 0; i < g_attr_n; ++i)
        if (g_attr[i].func == func && g_attr[i].device == dev) { slot = &g_attr[i]; break; }
    if (slot && slot->bytes >= bytes) return true;
    if (cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
        return false;
    if (!slot && g_attr_n < 256) slot = &g_attr[g_attr_n++];
    if (slot) { slot->func = func; slot->device = dev; slot->bytes = bytes; }
    return true;
}

}  // namespace swimba

// Host helper: build TMA tensor maps for bf16 tensors.  The driver entry point is looked up
// through the runtime so that the library does not link against libcuda directly.
#include "tc_host.cuh"

#include <cudaTypedefs.h>
#include <mutex>

namespace castling {
namespace tc {

namespace {
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
std::once_flag g_once;

void lookup() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
        g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
}

// A few recently built maps are kept: a serving loop calls with the same tensors and shapes over
// and over, and encoding five maps per forward costs more host time than the launches.
struct CacheEntry {
    bool valid = false;
    const void* base = nullptr;
    int rank = 0;
    uint64_t dims[5] = {};
    uint64_t strides[4] = {};
    uint32_t box[5] = {};
    bool swizzle = false;
    CUtensorMap map;
};
constexpr int kCacheSize = 32;
CacheEntry g_cache[kCacheSize];
int g_cache_next = 0;
std::mutex g_cache_mutex;

bool same_key(const CacheEntry& e, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
              const uint32_t* box, bool sw) {
    if (!e.valid || e.base != base || e.rank != rank || e.swizzle != sw) return false;
    for (int i = 0; i < rank; ++i)
        if (e.dims[i] != dims[i] || e.box[i] != box[i]) return false;
    for (int i = 0; i + 1 < rank; ++i)
        if (e.strides[i] != strides[i]) return false;
    return true;
}
}  // namespace

namespace {
bool encode_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides, const uint32_t* box, bool swizzle128);
}

// dims/box are innermost-first, in elements; the innermost dimension is contiguous; strides[i] is the
// distance in elements between consecutive indices of dimension i + 1 (rank - 1 entries).
bool make_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                          const uint64_t* strides, const uint32_t* box, bool swizzle128) {
    if (rank < 2 || rank > 5) return false;
    uint64_t fixed[4];
    for (int i = 0; i + 1 < rank; ++i) {
        fixed[i] = (dims[i + 1] == 1 && strides[i] == 0) ? 8 : strides[i];  // never stepped over: any legal value
        if (fixed[i] == 0 || (fixed[i] * 2) % 16 != 0 || fixed[i] * 2 >= (1ull << 40)) return false;
    }
    strides = fixed;
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    for (const CacheEntry& e : g_cache)
        if (same_key(e, base, rank, dims, strides, box, swizzle128)) { *out = e.map; return true; }
    if (!encode_tensor_map_bf16(out, base, rank, dims, strides, box, swizzle128)) return false;
    CacheEntry& e = g_cache[g_cache_next];
    g_cache_next = (g_cache_next + 1) % kCacheSize;
    e.valid = true; e.base = base; e.rank = rank; e.swizzle = swizzle128; e.map = *out;
    for (int i = 0; i < rank; ++i) { e.dims[i] = dims[i]; e.box[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) e.strides[i] = strides[i];
    return true;
}

namespace {
bool encode_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides, const uint32_t* box, bool swizzle128) {
    std::call_once(g_once, lookup);
    if (!g_encode) return false;
    cuuint64_t gdim[5];
    cuuint64_t gstride[4];
    cuuint32_t bdim[5], estride[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bdim[i] = box[i];
        estride[i] = 1;
        if (i + 1 < rank) gstride[i] = strides[i] * 2;  // bytes
    }
    const CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim,
                                gstride, bdim, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}
}  // namespace

}  // namespace tc
}  // namespace castling

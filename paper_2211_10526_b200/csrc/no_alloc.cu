// castling_attn_forward_static: the forward pass for callers that must not allocate device
// memory.  The partial and final d x d states that the state kernel hands to the apply kernel
// live in a fixed array in this library's device image instead of a cudaMalloc'd workspace.
#include "castling_attn.h"
#include "castling_internal.cuh"

#include <mutex>

namespace {

// 4 MiB of fp32 scratch per GPU that loads the library, held until the process exits.
constexpr size_t kStaticScratchWords = CASTLING_STATIC_SCRATCH_BYTES / sizeof(float);
static __device__ __align__(256) float g_static_scratch[kStaticScratchWords];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
float* g_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

// In host code `g_static_scratch` only names the symbol; its address on the device that is
// current has to be asked for.  Done once per device, on that device's first call.
int scratch_address(float** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return CASTLING_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return CASTLING_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { (void)cudaGetLastError(); return CASTLING_ERR_CUDA; }
        if (prop.major != 10) return CASTLING_ERR_ARCH;
        float* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return CASTLING_ERR_CUDA;
        }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return CASTLING_OK;
}

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
    return x < y + nb && y < x + na;
}

}  // namespace

extern "C" int castling_attn_forward_static(const void* q, const void* k, const void* v, const void* dw_weight,
                                            const void* dw_bias, void* out, int B, int H, int gridH, int gridW,
                                            int d, int ksize, double eps, castling_dtype_t dtype, void* stream) {
    if (!q || !k || !v || !dw_weight || !out) return CASTLING_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || gridH <= 0 || gridW <= 0 || d <= 0) return CASTLING_ERR_INVALID_ARG;
    if (ksize <= 0 || (ksize & 1) == 0) return CASTLING_ERR_INVALID_ARG;
    if (dtype != CASTLING_F32 && dtype != CASTLING_BF16) return CASTLING_ERR_UNSUPPORTED;
    if (!castling::simt_supports(d, ksize)) return CASTLING_ERR_UNSUPPORTED;
    const long long N = (long long)gridH * gridW, BH = (long long)B * H;
    if (N > (1 << 24) || BH > (1 << 20) || BH * ((N + 63) / 64) > 0x7fffffffLL) return CASTLING_ERR_UNSUPPORTED;
    const size_t eb = dtype == CASTLING_F32 ? 4 : 2;
    const size_t tensor_bytes = (size_t)BH * N * d * eb;
    const void* ptrs[4] = {q, k, v, out};
    for (const void* p : ptrs)
        if ((uintptr_t)p & 15) return CASTLING_ERR_ALIGNMENT;
    const size_t w_bytes = (size_t)H * d * ksize * ksize * eb, b_bytes = (size_t)H * d * eb;
    if (overlaps(out, tensor_bytes, q, tensor_bytes) || overlaps(out, tensor_bytes, k, tensor_bytes) ||
        overlaps(out, tensor_bytes, v, tensor_bytes) || overlaps(out, tensor_bytes, dw_weight, w_bytes) ||
        (dw_bias && overlaps(out, tensor_bytes, dw_bias, b_bytes)))
        return CASTLING_ERR_INVALID_ARG;

    // scratch: final state [BH][d*d + d], then (only if the token range is split) P partial states
    // per (b,h).  If the split version does not fit, fall back to one split; if that does not fit
    // either, the problem is beyond what this entry point serves.
    const size_t words = castling::state_words(d);
    int P = castling::simt_choose_splits((int)BH, (int)N);
    if ((size_t)BH * words * (1 + (P > 1 ? P : 0)) > kStaticScratchWords) P = 1;
    if ((size_t)BH * words > kStaticScratchWords) return CASTLING_ERR_SCRATCH_LIMIT;

    float* scratch = nullptr;
    const int rc = scratch_address(&scratch);
    if (rc != CASTLING_OK) return rc;

    castling::Problem p;
    p.q = q; p.k = k; p.v = v; p.w = dw_weight; p.bias = dw_bias; p.out = out;
    p.B = B; p.H = H; p.gridH = gridH; p.gridW = gridW; p.d = d; p.ksize = ksize;
    p.prefix = 0; p.N = (int)N; p.BH = (int)BH; p.head0 = 0;
    p.set_contiguous();
    p.bf16 = (dtype == CASTLING_BF16);
    if (eps <= 0.0) eps = 1e-12;
    p.eps2 = (float)(eps * eps);
    castling::KernelTimer timer;  // off: records nothing, creates nothing
    int launches = 0;
    // Nothing in the scratch has to start at zero: the state kernel overwrites every word that the
    // reduce and apply kernels read, so the previous call's contents are simply replaced.
    const cudaError_t e = castling::simt_forward(p, scratch, scratch + (size_t)BH * words, P,
                                                 static_cast<cudaStream_t>(stream), &launches, &timer);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return CASTLING_ERR_CUDA; }
    return CASTLING_OK;
}

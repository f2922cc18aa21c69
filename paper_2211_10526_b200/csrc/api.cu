// Host side of the C ABI declared in include/castling_attn.h: handle, argument
// validation, workspace, kernel-family dispatch.  No computation happens here.
#include "castling_attn.h"
#include "castling_internal.cuh"
#include "tc_host.cuh"

#include <new>

using castling::Problem;

struct castling_attn {
    castling_attn_config_t cfg;
    int device = 0;
    float* ws = nullptr;        // header | state | partial
    size_t ws_bytes = 0;
    unsigned* counters = nullptr;  // arrival counters of the split reduction, zero between calls
    size_t counters_cap = 0;
    char* stage = nullptr;      // device staging for castling_attn_forward_host
    size_t stage_bytes = 0;
    // castling_attn_forward_host pipelines batch chunks: copies in, kernels and copies out overlap
    static constexpr int kMaxChunks = 8;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_end = nullptr, ev_in[kMaxChunks] = {}, ev_done[kMaxChunks] = {};
    int last_cuda_error = 0;
    int last_path = 0;
    int last_launches = 0;
    castling::KernelTimer timer;
};

namespace castling {
int device_sm_count() {
    static std::atomic<int> cached[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { (void)cudaGetLastError(); return 148; }
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        return 148;
    }
    cached[dev].store(n, std::memory_order_relaxed);
    return n;
}
}  // namespace castling

namespace {

size_t elem_bytes(castling_dtype_t t) { return t == CASTLING_F32 ? 4 : 2; }

// header | state [BH] | partial [BH][P] (only when the token range is split)
size_t workspace_words(int BH, int N, int d, bool bf16) {
    int P = castling::simt_choose_splits(BH, N);
    size_t words = castling::state_words_rownorm(d);  // the CUDA-core kernels' state, with room for the key-row sum
    if (bf16 && (d == 64 || d == 32)) {  // shapes the tensor-core kernels may take: they keep 64-wide states
        const int Pt = castling::tc::choose_splits(BH, castling::tc::rows_per_head(N, d));
        if (Pt > P) P = Pt;
        if (castling::tc::kStateWordsRownorm > words) words = castling::tc::kStateWordsRownorm;
    }
    size_t slots = (size_t)BH * (P > 1 ? P : 0);  // partial states behind the BH final ones
    if (bf16 && d == 32 && BH % 2 == 0) {
        // two width-32 heads side by side (token-major layouts): BH / 2 planes of N rows each
        const int Pp = castling::tc::choose_splits(BH / 2, N);
        if (Pp > 1 && (size_t)(BH / 2) * Pp > slots) slots = (size_t)(BH / 2) * Pp;
    }
    size_t behind = slots * words;  // what follows the BH final states
    if (bf16 && (d == 64 || d == 32)) {  // the one-kernel forward keeps its per-plane operand blocks there
        const size_t r = castling::tc::pipe_ready_words(BH);
        if (r > behind) behind = r;
    }
    return castling::kHeaderWords + (size_t)BH * words + behind;
}

int fail_cuda(castling_attn* h, cudaError_t e, int code = CASTLING_ERR_CUDA) {
    if (h) h->last_cuda_error = (int)e;
    (void)cudaGetLastError();  // reset the runtime's last-error slot
    return code;
}

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
    return x < y + nb && y < x + na;
}

// Shape / dtype checks shared by the device- and host-pointer entry points.
int check_shape(const castling_attn* h, int B, int H, int gridH, int gridW, int d, castling_dtype_t dtype) {
    if (!h) return CASTLING_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || gridH <= 0 || gridW <= 0 || d <= 0) return CASTLING_ERR_INVALID_ARG;
    if (dtype != CASTLING_F32 && dtype != CASTLING_BF16) return CASTLING_ERR_UNSUPPORTED;
    if (!castling::simt_supports(d, h->cfg.ksize)) return CASTLING_ERR_UNSUPPORTED;
    const long long N = (long long)gridH * gridW + h->cfg.prefix_tokens, BH = (long long)B * H;
    if (N > (1 << 24) || BH > (1 << 20) || BH * ((N + 63) / 64) > 0x7fffffffLL) return CASTLING_ERR_UNSUPPORTED;
    if (BH * N * d > (1LL << 40)) return CASTLING_ERR_UNSUPPORTED;
    return CASTLING_OK;
}

int ensure_workspace(castling_attn* h, int BH, int N, int d, bool bf16) {
    const size_t need = workspace_words(BH, N, d, bf16) * sizeof(float);
    if (need <= h->ws_bytes) return CASTLING_OK;
    if (h->cfg.max_workspace && need > h->cfg.max_workspace) return CASTLING_ERR_OOM;
    cudaError_t e = cudaDeviceSynchronize();  // nothing may still be using the old buffer
    if (e != cudaSuccess) return fail_cuda(h, e);
    if (h->ws) cudaFree(h->ws);
    h->ws = nullptr; h->ws_bytes = 0;
    e = cudaMalloc((void**)&h->ws, need);
    if (e != cudaSuccess) return fail_cuda(h, e, CASTLING_ERR_OOM);
    e = cudaMemset(h->ws, 0, castling::kHeaderWords * sizeof(float));
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->ws_bytes = need;
    return CASTLING_OK;
}

int ensure_counters(castling_attn* h, int BH) {
    // either variant of the tensor-core path: 17 words per plane, or a header and 4 words per plane
    const size_t a = (size_t)BH * castling::tc::kCountersPerHead;
    const size_t b = castling::tc::kPipeCtrHeader + (size_t)BH * castling::tc::kPipeCtrPerPlane;
    const size_t want = a > b ? a : b;
    if (want <= h->counters_cap) return CASTLING_OK;
    size_t cap = 4096;
    while (cap < want) cap *= 2;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return fail_cuda(h, e);
    if (h->counters) cudaFree(h->counters);
    h->counters = nullptr; h->counters_cap = 0;
    e = cudaMalloc((void**)&h->counters, cap * sizeof(unsigned));
    if (e != cudaSuccess) return fail_cuda(h, e, CASTLING_ERR_OOM);
    e = cudaMemset(h->counters, 0, cap * sizeof(unsigned));
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->counters_cap = cap;
    return CASTLING_OK;
}

}  // namespace

extern "C" {

int castling_attn_create(const castling_attn_config_t* cfg, castling_attn_t** out_handle) {
    if (!out_handle) return CASTLING_ERR_INVALID_ARG;
    *out_handle = nullptr;
    castling_attn_config_t c = {3, 1e-12, CASTLING_PATH_AUTO, 0, 0, 0, 0, 0, 0.0};
    if (cfg) c = *cfg;
    if (c.eps <= 0.0) c.eps = 1e-12;
    if (c.ksize <= 0 || (c.ksize & 1) == 0) return CASTLING_ERR_INVALID_ARG;
    if (c.ksize > 7) return CASTLING_ERR_UNSUPPORTED;
    if (c.force_path < CASTLING_PATH_AUTO || c.force_path > CASTLING_PATH_TENSOR) return CASTLING_ERR_INVALID_ARG;
    if (c.prefix_tokens < 0) return CASTLING_ERR_INVALID_ARG;
    if (c.prefix_tokens > 16) return CASTLING_ERR_UNSUPPORTED;
    if ((c.normalize_rows | c.exact_kernel | c.sparse_branch) & ~1) return CASTLING_ERR_INVALID_ARG;
    if ((c.exact_kernel || c.sparse_branch) && c.prefix_tokens > 0) return CASTLING_ERR_UNSUPPORTED;
    if (c.sparse_branch && !(c.sparse_eps == c.sparse_eps)) return CASTLING_ERR_INVALID_ARG;  // NaN
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(nullptr, e);
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) return fail_cuda(nullptr, e);
    if (prop.major != 10) return CASTLING_ERR_ARCH;
    castling_attn* h = new (std::nothrow) castling_attn();
    if (!h) return CASTLING_ERR_OOM;
    h->cfg = c;
    h->device = dev;
    *out_handle = h;
    return CASTLING_OK;
}

int castling_attn_destroy(castling_attn_t* h) {
    if (!h) return CASTLING_OK;
    if (h->ws) cudaFree(h->ws);
    if (h->stage) cudaFree(h->stage);
    if (h->counters) cudaFree(h->counters);
    if (h->copy_in) cudaStreamDestroy(h->copy_in);
    if (h->copy_out) cudaStreamDestroy(h->copy_out);
    if (h->ev_start) cudaEventDestroy(h->ev_start);
    if (h->ev_end) cudaEventDestroy(h->ev_end);
    for (auto& e : h->ev_in) if (e) cudaEventDestroy(e);
    for (auto& e : h->ev_done) if (e) cudaEventDestroy(e);
    for (auto& e : h->timer.ev)
        if (e) cudaEventDestroy(e);
    delete h;
    return CASTLING_OK;
}

size_t castling_attn_workspace_bytes(int B, int H, int gridH, int gridW, int d, castling_dtype_t dtype) {
    if (B <= 0 || H <= 0 || gridH <= 0 || gridW <= 0 || d <= 0 || d > 128 || d % 16) return 0;
    if (dtype != CASTLING_F32 && dtype != CASTLING_BF16) return 0;
    return workspace_words(B * H, gridH * gridW, d, dtype == CASTLING_BF16) * sizeof(float);
}

const char* castling_attn_error_string(int code) {
    switch (code) {
        case CASTLING_OK: return "success";
        case CASTLING_ERR_INVALID_ARG: return "invalid argument (NULL pointer, non-positive size, even ksize or overlapping buffers)";
        case CASTLING_ERR_UNSUPPORTED: return "unsupported head width, filter size, dtype or problem size";
        case CASTLING_ERR_ALIGNMENT: return "tensor pointer is not 16-byte aligned";
        case CASTLING_ERR_ARCH: return "current CUDA device is not compute capability 10.x";
        case CASTLING_ERR_CUDA: return "a CUDA call failed (see castling_attn_last_cuda_error)";
        case CASTLING_ERR_OOM: return "workspace allocation failed or exceeds max_workspace";
        case CASTLING_ERR_DEVICE: return "a kernel gave up on a bounded wait";
        case CASTLING_ERR_SCRATCH_LIMIT: return "problem needs more than the library's static scratch (use castling_attn_forward with a handle)";
        default: return "unknown castling_attn error code";
    }
}

int castling_attn_last_cuda_error(const castling_attn_t* h) { return h ? h->last_cuda_error : 0; }

int castling_attn_last_path(const castling_attn_t* h, int* kernel_launches) {
    if (!h) return CASTLING_ERR_INVALID_ARG;
    if (kernel_launches) *kernel_launches = h->last_launches;
    return h->last_path;
}

}  // extern "C"

namespace {

// Enqueue the kernels for one validated problem whose tensors are all on the device.
int run_device(castling_attn* h, const Problem& p, cudaStream_t stream) {
    if (p.exact_kernel || p.sparse) {
        // explicit attention weights: one kernel, no workspace; quadratic in the number of tokens
        if (p.N > 16384) return CASTLING_ERR_UNSUPPORTED;
        const bool tensor_quad = castling::tc::quad_supports(p) && h->cfg.force_path != CASTLING_PATH_SIMT;
        if (h->cfg.force_path == CASTLING_PATH_TENSOR && !tensor_quad) return CASTLING_ERR_UNSUPPORTED;
        int launches = 0;
        h->timer.begin(stream);
        if (tensor_quad) {
            // the exact kernel alone on bf16 heads of width 64: cosines and weighted sums on the tensor cores
            const int rc = ensure_workspace(h, 1, 64, 64, true);  // the status word lives at the head of the workspace
            if (rc != CASTLING_OK) return rc;
            const cudaError_t eq = castling::tc::launch_quad(p, reinterpret_cast<unsigned*>(h->ws), stream);
            if (eq == cudaSuccess) {
                h->timer.mark(stream, "tc_quad");
                h->last_path = CASTLING_PATH_TENSOR;
                h->last_launches = 1;
                return CASTLING_OK;
            }
            if (eq != cudaErrorNotSupported || h->cfg.force_path == CASTLING_PATH_TENSOR) return fail_cuda(h, eq);
            (void)cudaGetLastError();  // strides the tensor maps cannot take: the CUDA-core kernel takes any layout
            h->timer.begin(stream);
        }
        const cudaError_t e = castling::quad_forward(p, stream, &launches, &h->timer);
        if (e == cudaErrorNotSupported) { (void)cudaGetLastError(); return CASTLING_ERR_UNSUPPORTED; }
        if (e != cudaSuccess) return fail_cuda(h, e);
        h->last_path = CASTLING_PATH_SIMT;
        h->last_launches = launches;
        return CASTLING_OK;
    }
    int rc = ensure_workspace(h, p.BH, p.N, p.d, p.bf16);
    if (rc != CASTLING_OK) return rc;
    const bool tensor_ok = castling::tc::supports(p);
    if (h->cfg.force_path == CASTLING_PATH_TENSOR && !tensor_ok) return CASTLING_ERR_UNSUPPORTED;
    bool use_tensor = tensor_ok && (h->cfg.force_path == CASTLING_PATH_TENSOR ||
                                    (h->cfg.force_path == CASTLING_PATH_AUTO && castling::tc::preferred(p)));
    float* state = h->ws + castling::kHeaderWords;
    const size_t simt_words = p.rownorm ? castling::state_words_rownorm(p.d) : castling::state_words(p.d);
    float* partial = state + (size_t)p.BH * (use_tensor ? (size_t)castling::tc::state_words_of(p) : simt_words);
    int launches = 0;
    h->timer.begin(stream);
    cudaError_t e;
    if (use_tensor) {
        rc = ensure_counters(h, p.BH);
        if (rc != CASTLING_OK) return rc;
        e = castling::tc::forward(p, state, partial, h->counters, castling::tc::choose_splits(p.BH, castling::tc::rows_per_head(p.N, p.d)),
                                  reinterpret_cast<unsigned*>(h->ws), stream, &launches, &h->timer);
    } else {
        e = castling::simt_forward(p, state, partial, castling::simt_choose_splits(p.BH, p.N), stream, &launches,
                                   &h->timer);
    }
    if (use_tensor && e == cudaErrorNotSupported && h->cfg.force_path == CASTLING_PATH_AUTO) {
        // the TMA descriptor could not be encoded for these strides: the CUDA-core kernels take any layout
        (void)cudaGetLastError();
        use_tensor = false;
        partial = state + (size_t)p.BH * simt_words;
        h->timer.begin(stream);
        e = castling::simt_forward(p, state, partial, castling::simt_choose_splits(p.BH, p.N), stream, &launches, &h->timer);
    }
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->last_path = use_tensor ? CASTLING_PATH_TENSOR : CASTLING_PATH_SIMT;
    h->last_launches = launches;
    return CASTLING_OK;
}

Problem make_problem(const castling_attn* h, const void* q, const void* k, const void* v, const void* w,
                     const void* bias, void* out, int B, int H, int gridH, int gridW, int d,
                     castling_dtype_t dtype) {
    Problem p;
    p.q = q; p.k = k; p.v = v; p.w = w; p.bias = bias; p.out = out;
    p.B = B; p.H = H; p.gridH = gridH; p.gridW = gridW; p.d = d; p.ksize = h->cfg.ksize;
    p.prefix = h->cfg.prefix_tokens;
    p.N = p.prefix + gridH * gridW; p.BH = B * H; p.head0 = 0;
    p.bf16 = (dtype == CASTLING_BF16);
    p.eps2 = (float)(h->cfg.eps * h->cfg.eps);
    p.rownorm = h->cfg.normalize_rows != 0;
    p.exact_kernel = h->cfg.exact_kernel != 0;
    p.sparse = h->cfg.sparse_branch != 0;
    p.sparse_eps = (float)h->cfg.sparse_eps;
    p.set_contiguous();
    return p;
}

// Elements spanned by a [B, H, N, d] tensor laid out with the given strides.
long long extent(long long batch, long long head, long long token, int B, int H, long long N, int d) {
    return (B - 1) * batch + (H - 1) * head + (N - 1) * token + d;
}

}  // namespace

extern "C" {

int castling_attn_forward(castling_attn_t* h, const void* q, const void* k, const void* v,
                          const void* dw_weight, const void* dw_bias, void* out,
                          int B, int H, int gridH, int gridW, int d, castling_dtype_t dtype, void* stream) {
    int rc = check_shape(h, B, H, gridH, gridW, d, dtype);
    if (rc != CASTLING_OK) return rc;
    if (!q || !k || !v || !dw_weight || !out) return CASTLING_ERR_INVALID_ARG;
    const size_t eb = elem_bytes(dtype);
    const size_t tensor_bytes = (size_t)B * H * (h->cfg.prefix_tokens + (size_t)gridH * gridW) * d * eb;
    const size_t w_bytes = (size_t)H * d * h->cfg.ksize * h->cfg.ksize * eb;
    const size_t b_bytes = (size_t)H * d * eb;
    const void* ptrs[4] = {q, k, v, out};
    for (const void* ptr : ptrs)
        if ((uintptr_t)ptr & 15) return CASTLING_ERR_ALIGNMENT;
    if (overlaps(out, tensor_bytes, q, tensor_bytes) || overlaps(out, tensor_bytes, k, tensor_bytes) ||
        overlaps(out, tensor_bytes, v, tensor_bytes) || overlaps(out, tensor_bytes, dw_weight, w_bytes) ||
        (dw_bias && overlaps(out, tensor_bytes, dw_bias, b_bytes)))
        return CASTLING_ERR_INVALID_ARG;
    const Problem p = make_problem(h, q, k, v, dw_weight, dw_bias, out, B, H, gridH, gridW, d, dtype);
    return run_device(h, p, static_cast<cudaStream_t>(stream));
}

int castling_attn_forward_strided(castling_attn_t* h, const void* q, const void* k, const void* v,
                                  const void* dw_weight, const void* dw_bias, void* out,
                                  int B, int H, int gridH, int gridW, int d, castling_dtype_t dtype,
                                  const castling_attn_layout_t* layout, void* stream) {
    int rc = check_shape(h, B, H, gridH, gridW, d, dtype);
    if (rc != CASTLING_OK) return rc;
    if (!q || !k || !v || !dw_weight || !out || !layout) return CASTLING_ERR_INVALID_ARG;
    const long long eb = (long long)elem_bytes(dtype), N = (long long)gridH * gridW + h->cfg.prefix_tokens;
    const long long* s = &layout->q_batch;  // twelve strides: q, k, v, out x (batch, head, token)
    long long ext[4];
    for (int t = 0; t < 4; ++t) {
        const long long sb = s[3 * t], sh = s[3 * t + 1], st = s[3 * t + 2];
        if (sb < 0 || sh < 0 || st < d) return CASTLING_ERR_INVALID_ARG;
        if ((B > 1 && sb == 0) || (H > 1 && sh == 0)) return CASTLING_ERR_INVALID_ARG;
        if ((sb * eb) % 16 || (sh * eb) % 16 || (st * eb) % 16) return CASTLING_ERR_ALIGNMENT;
        if (sb > (1LL << 40) || sh > (1LL << 40) || st > (1LL << 32)) return CASTLING_ERR_UNSUPPORTED;
        ext[t] = extent(sb, sh, st, B, H, N, d);
        if (ext[t] > (1LL << 42)) return CASTLING_ERR_UNSUPPORTED;
    }
    const void* ptrs[4] = {q, k, v, out};
    for (const void* ptr : ptrs)
        if ((uintptr_t)ptr & 15) return CASTLING_ERR_ALIGNMENT;
    const size_t w_bytes = (size_t)H * d * h->cfg.ksize * h->cfg.ksize * eb, b_bytes = (size_t)H * d * eb;
    const size_t out_bytes = (size_t)(ext[3] * eb);
    if (overlaps(out, out_bytes, q, (size_t)(ext[0] * eb)) || overlaps(out, out_bytes, k, (size_t)(ext[1] * eb)) ||
        overlaps(out, out_bytes, v, (size_t)(ext[2] * eb)) || overlaps(out, out_bytes, dw_weight, w_bytes) ||
        (dw_bias && overlaps(out, out_bytes, dw_bias, b_bytes)))
        return CASTLING_ERR_INVALID_ARG;
    Problem p = make_problem(h, q, k, v, dw_weight, dw_bias, out, B, H, gridH, gridW, d, dtype);
    p.lq = {layout->q_batch, layout->q_head, layout->q_token};
    p.lk = {layout->k_batch, layout->k_head, layout->k_token};
    p.lv = {layout->v_batch, layout->v_head, layout->v_token};
    p.lo = {layout->out_batch, layout->out_head, layout->out_token};
    p.hdiv = H;
    return run_device(h, p, static_cast<cudaStream_t>(stream));
}

int castling_attn_forward_host(castling_attn_t* h, const void* q, const void* k, const void* v,
                               const void* dw_weight, const void* dw_bias, void* out,
                               int B, int H, int gridH, int gridW, int d, castling_dtype_t dtype, void* stream) {
    int rc = check_shape(h, B, H, gridH, gridW, d, dtype);
    if (rc != CASTLING_OK) return rc;
    if (!q || !k || !v || !dw_weight || !out) return CASTLING_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t eb = elem_bytes(dtype);
    const size_t n_tok = h->cfg.prefix_tokens + (size_t)gridH * gridW;
    const size_t tb = (((size_t)B * H * n_tok * d * eb) + 255) & ~(size_t)255;
    const size_t wb = (((size_t)H * d * h->cfg.ksize * h->cfg.ksize * eb) + 255) & ~(size_t)255;
    const size_t bb = (((size_t)H * d * eb) + 255) & ~(size_t)255;
    const size_t need = 4 * tb + wb + bb;
    if (need > h->stage_bytes) {
        if (h->cfg.max_workspace && need > h->cfg.max_workspace) return CASTLING_ERR_OOM;
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess) return fail_cuda(h, e);
        if (h->stage) cudaFree(h->stage);
        h->stage = nullptr; h->stage_bytes = 0;
        e = cudaMalloc((void**)&h->stage, need);
        if (e != cudaSuccess) return fail_cuda(h, e, CASTLING_ERR_OOM);
        h->stage_bytes = need;
    }
    char* dq = h->stage; char* dk = dq + tb; char* dv = dk + tb; char* dout = dv + tb;
    char* dw = dout + tb; char* db = dw + wb;
    const size_t t_exact = (size_t)B * H * n_tok * d * eb;
    cudaError_t e;
    if ((e = cudaMemcpyAsync(dw, dw_weight, (size_t)H * d * h->cfg.ksize * h->cfg.ksize * eb,
                             cudaMemcpyHostToDevice, st)) != cudaSuccess) return fail_cuda(h, e);
    if (dw_bias &&
        (e = cudaMemcpyAsync(db, dw_bias, (size_t)H * d * eb, cudaMemcpyHostToDevice, st)) != cudaSuccess)
        return fail_cuda(h, e);

    // Chunks of whole (b,h) planes, at least 8 MB of one tensor each: small problems go through in one piece.
    const int BH = B * H;
    const size_t plane_bytes = t_exact / BH;
    int chunks = BH < castling_attn::kMaxChunks ? BH : castling_attn::kMaxChunks;
    while (chunks > 1 && t_exact / chunks < ((size_t)8 << 20)) --chunks;
    if (chunks <= 1) {
        if ((e = cudaMemcpyAsync(dq, q, t_exact, cudaMemcpyHostToDevice, st)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaMemcpyAsync(dk, k, t_exact, cudaMemcpyHostToDevice, st)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaMemcpyAsync(dv, v, t_exact, cudaMemcpyHostToDevice, st)) != cudaSuccess) return fail_cuda(h, e);
        const Problem p = make_problem(h, dq, dk, dv, dw, dw_bias ? db : nullptr, dout, B, H, gridH, gridW, d, dtype);
        rc = run_device(h, p, st);
        if (rc != CASTLING_OK) return rc;
        if ((e = cudaMemcpyAsync(out, dout, t_exact, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return fail_cuda(h, e);
        return CASTLING_OK;
    }

    // Pipeline: all chunk uploads queue on a copy stream; the kernels of chunk c wait for its upload on the
    // caller's stream; its download runs on a second copy stream while later chunks upload and compute
    // (PCIe is full duplex).  Streams and events are created on first use and kept in the handle.
    if (!h->copy_in) {
        if ((e = cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaEventCreateWithFlags(&h->ev_end, cudaEventDisableTiming)) != cudaSuccess) return fail_cuda(h, e);
        for (int c = 0; c < castling_attn::kMaxChunks; ++c) {
            if ((e = cudaEventCreateWithFlags(&h->ev_in[c], cudaEventDisableTiming)) != cudaSuccess) return fail_cuda(h, e);
            if ((e = cudaEventCreateWithFlags(&h->ev_done[c], cudaEventDisableTiming)) != cudaSuccess) return fail_cuda(h, e);
        }
    }
    // the copy streams start after everything already queued on the caller's stream (filters included)
    if ((e = cudaEventRecord(h->ev_start, st)) != cudaSuccess) return fail_cuda(h, e);
    if ((e = cudaStreamWaitEvent(h->copy_in, h->ev_start, 0)) != cudaSuccess) return fail_cuda(h, e);
    if ((e = cudaStreamWaitEvent(h->copy_out, h->ev_start, 0)) != cudaSuccess) return fail_cuda(h, e);
    int b0[castling_attn::kMaxChunks + 1];
    for (int c = 0; c <= chunks; ++c) b0[c] = (int)((long long)BH * c / chunks);
    // workspace and counters for every run length, before anything is in flight: growing them later
    // would synchronise the device in the middle of the pipeline (and clear the status word)
    for (int c = 0; c < chunks; ++c) {
        rc = ensure_workspace(h, b0[c + 1] - b0[c], (int)n_tok, d, dtype == CASTLING_BF16);
        if (rc != CASTLING_OK) return rc;
        rc = ensure_counters(h, b0[c + 1] - b0[c]);
        if (rc != CASTLING_OK) return rc;
    }
    for (int c = 0; c < chunks; ++c) {
        const size_t off = (size_t)b0[c] * plane_bytes, len = (size_t)(b0[c + 1] - b0[c]) * plane_bytes;
        const char* hq = static_cast<const char*>(q); const char* hk = static_cast<const char*>(k);
        const char* hv = static_cast<const char*>(v);
        // K and V first: the state kernel needs them before the apply kernel needs Q
        if ((e = cudaMemcpyAsync(dk + off, hk + off, len, cudaMemcpyHostToDevice, h->copy_in)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaMemcpyAsync(dv + off, hv + off, len, cudaMemcpyHostToDevice, h->copy_in)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaMemcpyAsync(dq + off, hq + off, len, cudaMemcpyHostToDevice, h->copy_in)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaEventRecord(h->ev_in[c], h->copy_in)) != cudaSuccess) return fail_cuda(h, e);
    }
    for (int c = 0; c < chunks; ++c) {
        const size_t off = (size_t)b0[c] * plane_bytes, len = (size_t)(b0[c + 1] - b0[c]) * plane_bytes;
        if ((e = cudaStreamWaitEvent(st, h->ev_in[c], 0)) != cudaSuccess) return fail_cuda(h, e);
        Problem p = make_problem(h, dq + off, dk + off, dv + off, dw, dw_bias ? db : nullptr, dout + off,
                                 1, H, gridH, gridW, d, dtype);
        p.BH = b0[c + 1] - b0[c];   // a run of planes that may start and end inside a batch
        p.head0 = b0[c] % H;
        p.set_contiguous();         // one uniform plane stride over the run (planes per step = the run's length)
        rc = run_device(h, p, st);
        if (rc != CASTLING_OK) return rc;
        if ((e = cudaEventRecord(h->ev_done[c], st)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaStreamWaitEvent(h->copy_out, h->ev_done[c], 0)) != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaMemcpyAsync(static_cast<char*>(out) + off, dout + off, len, cudaMemcpyDeviceToHost, h->copy_out)) != cudaSuccess)
            return fail_cuda(h, e);
    }
    if ((e = cudaEventRecord(h->ev_end, h->copy_out)) != cudaSuccess) return fail_cuda(h, e);
    if ((e = cudaStreamWaitEvent(st, h->ev_end, 0)) != cudaSuccess) return fail_cuda(h, e);
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return fail_cuda(h, e);
    return CASTLING_OK;
}

int castling_attn_device_status(castling_attn_t* h, void* stream, unsigned int* raw) {
    if (!h) return CASTLING_ERR_INVALID_ARG;
    unsigned int word = 0;
    if (h->ws) {
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        cudaError_t e = cudaMemcpyAsync(&word, h->ws, sizeof(word), cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return fail_cuda(h, e);
        if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return fail_cuda(h, e);
    }
    if (raw) *raw = word;
    if (word) {
        // reported once: the word is cleared, and so are arrival counters that a kernel which gave up may have
        // left half way
        cudaMemset(h->ws, 0, sizeof(unsigned));
        if (h->counters) cudaMemset(h->counters, 0, h->counters_cap * sizeof(unsigned));
    }
    return word ? CASTLING_ERR_DEVICE : CASTLING_OK;
}

size_t castling_attn_state_words(int d) { return d > 0 ? castling::state_words(d) : 0; }

// The two halves of a forward whose token grid is cut into bands of rows held by different devices.
static int shard_config_ok(const castling_attn* h) {
    if (!h) return CASTLING_ERR_INVALID_ARG;
    if (h->cfg.prefix_tokens || h->cfg.normalize_rows || h->cfg.exact_kernel || h->cfg.sparse_branch) return CASTLING_ERR_UNSUPPORTED;
    return CASTLING_OK;
}

int castling_attn_shard_state(castling_attn_t* h, const void* k, const void* v, float* state_out,
                              int B, int H, int n_tokens, int d, castling_dtype_t dtype, void* stream) {
    int rc = shard_config_ok(h);
    if (rc != CASTLING_OK) return rc;
    rc = check_shape(h, B, H, 1, n_tokens, d, dtype);
    if (rc != CASTLING_OK) return rc;
    if (!k || !v || !state_out) return CASTLING_ERR_INVALID_ARG;
    if (((uintptr_t)k | (uintptr_t)v | (uintptr_t)state_out) & 15) return CASTLING_ERR_ALIGNMENT;
    Problem p = make_problem(h, nullptr, k, v, nullptr, nullptr, nullptr, B, H, 1, n_tokens, d, dtype);
    p.phase = castling::kPhaseStateOnly;
    rc = ensure_workspace(h, p.BH, p.N, p.d, p.bf16);
    if (rc != CASTLING_OK) return rc;
    float* partial = h->ws + castling::kHeaderWords + (size_t)p.BH * castling::state_words(p.d);
    int launches = 0;
    h->timer.begin(static_cast<cudaStream_t>(stream));
    bool tensor = h->cfg.force_path != CASTLING_PATH_SIMT && castling::tc::shard_supports(p);
    cudaError_t e = cudaSuccess;
    if (tensor) {
        rc = ensure_counters(h, p.BH);
        if (rc != CASTLING_OK) return rc;
        // the partial states of the tensor-core kernel follow BH final-state slots of its own size
        partial = h->ws + castling::kHeaderWords + (size_t)p.BH * castling::tc::kStateWords;
        e = castling::tc::shard_state(p, state_out, partial, h->counters, reinterpret_cast<unsigned*>(h->ws),
                                      static_cast<cudaStream_t>(stream), &launches, &h->timer);
        if (e == cudaErrorNotSupported) { (void)cudaGetLastError(); tensor = false; h->timer.begin(static_cast<cudaStream_t>(stream)); }
    }
    if (!tensor) {
        partial = h->ws + castling::kHeaderWords + (size_t)p.BH * castling::state_words(p.d);
        e = castling::simt_forward(p, state_out, partial, castling::simt_choose_splits(p.BH, p.N),
                                   static_cast<cudaStream_t>(stream), &launches, &h->timer);
    }
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->last_path = tensor ? CASTLING_PATH_TENSOR : CASTLING_PATH_SIMT; h->last_launches = launches;
    return CASTLING_OK;
}

int castling_attn_shard_apply(castling_attn_t* h, const void* q, const void* v_halo, const void* dw_weight,
                              const void* dw_bias, const float* state, void* out, int B, int H, int gridH_local,
                              int gridW, int halo_top, int halo_bottom, int d, castling_dtype_t dtype, void* stream) {
    int rc = shard_config_ok(h);
    if (rc != CASTLING_OK) return rc;
    rc = check_shape(h, B, H, gridH_local, gridW, d, dtype);
    if (rc != CASTLING_OK) return rc;
    if (!q || !v_halo || !dw_weight || !state || !out) return CASTLING_ERR_INVALID_ARG;
    const int r = (h->cfg.ksize - 1) / 2;
    if (halo_top < 0 || halo_bottom < 0 || halo_top > r || halo_bottom > r) return CASTLING_ERR_INVALID_ARG;
    if (((uintptr_t)q | (uintptr_t)v_halo | (uintptr_t)out | (uintptr_t)state) & 15) return CASTLING_ERR_ALIGNMENT;
    Problem p = make_problem(h, q, nullptr, v_halo, dw_weight, dw_bias, out, B, H, gridH_local, gridW, d, dtype);
    p.phase = castling::kPhaseApplyOnly;
    p.v_row0 = halo_top;
    p.v_rows = halo_top + gridH_local + halo_bottom;
    p.lv.head = (long long)p.v_rows * gridW * d;   // planes of the taller V tensor
    int launches = 0;
    h->timer.begin(static_cast<cudaStream_t>(stream));
    bool tensor = h->cfg.force_path != CASTLING_PATH_SIMT && castling::tc::shard_supports(p);
    cudaError_t e = cudaSuccess;
    if (tensor) {
        rc = ensure_workspace(h, 1, 64, 64, true);  // the status word lives at the head of the workspace
        if (rc != CASTLING_OK) return rc;
        e = castling::tc::shard_apply(p, state, reinterpret_cast<unsigned*>(h->ws), static_cast<cudaStream_t>(stream),
                                      &launches, &h->timer);
        if (e == cudaErrorNotSupported) { (void)cudaGetLastError(); tensor = false; h->timer.begin(static_cast<cudaStream_t>(stream)); }
    }
    if (!tensor)
        e = castling::simt_forward(p, const_cast<float*>(state), nullptr, 1, static_cast<cudaStream_t>(stream), &launches,
                                   &h->timer);
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->last_path = tensor ? CASTLING_PATH_TENSOR : CASTLING_PATH_SIMT; h->last_launches = launches;
    return CASTLING_OK;
}

int castling_attn_selftest_wait(castling_attn_t* h, unsigned int limit_us, void* stream) {
    if (!h || limit_us == 0 || limit_us > 1000000u) return CASTLING_ERR_INVALID_ARG;
    int rc = ensure_workspace(h, 1, 64, 64, true);  // the status word lives at the head of the workspace
    if (rc != CASTLING_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned* status = reinterpret_cast<unsigned*>(h->ws);
    unsigned* reached = status + 1;  // header word 1 is free
    cudaError_t e = cudaMemsetAsync(reached, 0, sizeof(unsigned), st);
    if (e != cudaSuccess) return fail_cuda(h, e);
    e = castling::tc::launch_selftest_wait(status, (unsigned long long)limit_us * 1000ull, reached, st);
    if (e != cudaSuccess) return fail_cuda(h, e);
    unsigned end = 0;
    if ((e = cudaMemcpyAsync(&end, reached, sizeof(end), cudaMemcpyDeviceToHost, st)) != cudaSuccess) return fail_cuda(h, e);
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return fail_cuda(h, e);
    return end == 1u ? CASTLING_OK : CASTLING_ERR_DEVICE;  // 1: the kernel ran to its end after the wait gave up
}

int castling_attn_set_profiling(castling_attn_t* h, int enable) {
    if (!h) return CASTLING_ERR_INVALID_ARG;
    h->timer.on = enable != 0;
    h->timer.n = 0;
    return CASTLING_OK;
}

int castling_attn_kernel_times(castling_attn_t* h, float* ms, const char** names, int capacity) {
    if (!h || capacity < 0 || (capacity > 0 && !ms)) return CASTLING_ERR_INVALID_ARG;
    if (!h->timer.on || h->timer.n == 0) return 0;
    cudaError_t e = cudaEventSynchronize(h->timer.ev[h->timer.n]);
    if (e != cudaSuccess) return fail_cuda(h, e);
    const int n = h->timer.n < capacity ? h->timer.n : capacity;
    for (int i = 0; i < n; ++i) {
        e = cudaEventElapsedTime(&ms[i], h->timer.ev[i], h->timer.ev[i + 1]);
        if (e != cudaSuccess) return fail_cuda(h, e);
        if (names) names[i] = h->timer.name[i];
    }
    return n;
}

}  // extern "C"

// Internal declarations shared by the host dispatcher and the kernel files of
// the linear-angular attention library.  Not part of the public ABI.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <atomic>
#include <stddef.h>
#include <stdint.h>

namespace castling {

constexpr float kInvPi = 0.31830988618379067154f;
constexpr int kPhaseAll = 0, kPhaseStateOnly = 1, kPhaseApplyOnly = 2;

// Element strides of one [B, H, N, d] tensor whose d elements are contiguous.
struct Layout {
    long long batch, head, token;
};

// Offset (in elements) of (b,h) plane i: planes are numbered b * hdiv + h with hdiv planes per batch step.
__host__ __device__ inline long long plane_offset(const Layout& l, int i, int hdiv) {
    const int b = i / hdiv;
    return (long long)b * l.batch + (long long)(i - b * hdiv) * l.head;
}

// One forward call, as the kernels see it.
struct Problem {
    const void* q;
    const void* k;
    const void* v;
    const void* w;     // [H*d, ksize, ksize]
    const void* bias;  // [H*d] or nullptr
    void* out;
    int B, H, gridH, gridW, d, ksize;
    int prefix = 0;    // leading off-grid tokens (class tokens): attended like the rest, not convolved
    int N;             // tokens per sequence: prefix + gridH * gridW
    int BH;            // B * H (the (b,h) planes of this call)
    int head0;         // head index of plane 0: plane i uses the filters of head (head0 + i) % H
    bool bf16;
    float eps2;        // eps^2: the floor under the sum of squares
    Layout lq, lk, lv, lo;  // where token n of plane i of q, k, v, out starts: plane_offset(l, i, hdiv) + n * l.token
    bool blockdiag = false;  // tensor-core path only: a width-64 plane holds two independent width-32 heads side by
                             // side (heads h, h+1 of a layout whose head stride is 32): rows are normalised per
                             // half and only the two diagonal 32 x 32 blocks of the state are used
    // Variants beyond the inference-time core (all off by default):
    bool rownorm = false;       // every row of attention weights divided by its sum (Eq. 3's denominator)
    bool exact_kernel = false;  // 1 - arccos(x)/pi (Eq. 4-5) instead of its kept part 1/2 + x/pi (Eq. 8)
    bool sparse = false;        // plus Mask_eps(Softmax(q^ k^^T)) (Eq. 10)
    float sparse_eps = 0.f;     // the mask's threshold
    // A forward cut in two for sequences sharded over devices (CUDA-core kernels): the state of this shard's tokens
    // only, or the apply pass only with a state summed over all shards given in the workspace's place.
    int phase = 0;              // kPhaseAll / kPhaseStateOnly / kPhaseApplyOnly
    int v_row0 = 0, v_rows = 0; // apply of a shard: V holds v_rows grid rows and its row v_row0 is the shard's row 0
                                // (v_rows = 0: V holds exactly the gridH rows)
    int hdiv;          // planes per batch step of the layouts: H for a caller's strided tensors, BH for a
                       // run of contiguous planes (one uniform plane stride)
    // Contiguous [planes][N][d] tensors; needs N, d and BH.
    void set_contiguous() {
        const Layout c = {0, (long long)N * d, (long long)d};
        lq = lk = lv = lo = c;
        hdiv = BH;
    }
    bool contiguous_tokens() const { return lq.token == d && lk.token == d && lv.token == d && lo.token == d; }
};

// Workspace layout (fp32 words):
//   [0, 64)                          header; word 0 is the device status word
//   state  [BH][d*d + d]             raw sums: S = sum_n k^_n^T v_n, then s = sum_n v_n
//   partial[BH][P][d*d + d]          per-split sums when the token range is split P ways
constexpr size_t kHeaderWords = 64;

inline size_t state_words(int d) { return (size_t)d * d + d; }
// With row-sum normalisation the sum of the unit key rows follows: S, s, then sum_n k^_n (d more words).
inline size_t state_words_rownorm(int d) { return (size_t)d * d + 2 * (size_t)d; }

// Optional per-kernel timing: when `on`, an event is recorded on the stream before the first
// kernel of a forward and after every kernel, so the host can read each kernel's duration.
struct KernelTimer {
    static constexpr int kMax = 8;
    bool on = false;
    int n = 0;                       // kernels recorded by the most recent forward
    cudaEvent_t ev[kMax + 1] = {};   // created lazily
    const char* name[kMax] = {};
    void begin(cudaStream_t st) {
        n = 0;
        if (!on) return;
        if (!ev[0]) for (auto& e : ev) cudaEventCreate(&e);
        cudaEventRecord(ev[0], st);
    }
    void mark(cudaStream_t st, const char* kernel_name) {
        if (!on || n >= kMax) return;
        name[n] = kernel_name;
        cudaEventRecord(ev[++n], st);
    }
};

// Opt-in to more than 48 KiB of dynamic shared memory.  The attribute belongs to a kernel on one
// device, so it is set once per (kernel, device): `flags` is a static of the call site, one per kernel.
constexpr int kMaxDevices = 64;
struct PerDevice { std::atomic<bool> done[kMaxDevices]; };
template <typename Kernel>
inline cudaError_t opt_in_smem(Kernel kernel, size_t bytes, PerDevice& flags) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool tracked = dev >= 0 && dev < kMaxDevices;
    if (tracked && flags.done[dev].load(std::memory_order_acquire)) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && tracked) flags.done[dev].store(true, std::memory_order_release);
    return e;
}

// Multiprocessors of the current device (queried once per device).  Without a usable device the count
// of a B200 is returned, so that size queries still answer on a host without a GPU.
int device_sm_count();

// CUDA-core path.  simt_forward returns the cudaError_t of its launches.
cudaError_t simt_forward(const Problem& p, float* ws_state, float* ws_partial, int P,
                         cudaStream_t stream, int* launches, KernelTimer* timer);
int simt_choose_splits(int BH, int N);
// Explicit-weights forward (csrc/quad_kernels.cu): exact kernel and / or masked softmax branch; O(N^2 d).
cudaError_t quad_forward(const Problem& p, cudaStream_t stream, int* launches, KernelTimer* timer);
bool simt_supports(int d, int ksize);

}  // namespace castling

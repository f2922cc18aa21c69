/*
 * castling_attn.h -- C ABI of the linear-angular attention core for NVIDIA B200 (sm_100a).
 *
 * The library computes, for every batch b and head h independently, the
 * inference-time attention of Castling-ViT (arXiv 2211.10526, Sec. 3.2.1):
 *
 *     out_t = 1/2 * sum_j v_j  +  (1/pi) * q^_t (K^^T V)  +  DWConv(V)_t
 *
 * where q^_t = q_t / max(||q_t||_2, eps) and k^_j likewise are the unit rows the
 * paper prescribes for Q and K (text after Eq. 8; last sentence of Sec. 3.2.1),
 * 1/2 + (q^_t . k^_j)/pi is the kept "linear-angular" part of the expanded
 * angular kernel (Eq. 8), the product is re-associated so that only the d x d
 * state K^^T V and the token sum of V are formed (Eq. 9 and the "kernel-based
 * linear attention" paragraph of Sec. 3.1), and DWConv is the learnable
 * depthwise convolution applied to the value tokens on their 2-D grid
 * (Eq. 9, term M_DW V).  The masked softmax branch of Eq. 9-10 is all zeros at
 * inference (Sec. 3.2.2, "Castling during ViT inference") and is not computed.
 *
 * No row-sum denominator and no 1/sqrt(d) factor appear in Eq. 8-9, and none
 * is applied.  V is used as given.  The convolution is a cross-correlation
 * with zero "same" padding and stride 1, one ksize x ksize filter per
 * head-channel ch = h*d + j, plus an optional bias.
 *
 * All tensor arguments are plain pointers; nothing here depends on PyTorch.
 * Nothing in this library runs the computation on the CPU: without a CUDA
 * device of compute capability 10.x every forward call returns an error.
 */
#ifndef CASTLING_ATTN_H_
#define CASTLING_ATTN_H_

#include <stddef.h>

#if defined(__GNUC__)
#define CASTLING_API __attribute__((visibility("default")))
#else
#define CASTLING_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct castling_attn castling_attn_t; /* opaque handle */

typedef enum {
    CASTLING_F32 = 0, /* fp32 in, fp32 arithmetic, fp32 out                      */
    CASTLING_BF16 = 1 /* bf16 in, fp32 accumulation (bf16 tensor-core operands), */
                      /* one round-to-nearest-even to bf16 at the store          */
} castling_dtype_t;

/* Return codes.  0 is success; everything else is negative. */
enum {
    CASTLING_OK = 0,
    CASTLING_ERR_INVALID_ARG = -1, /* NULL pointer, non-positive size, even ksize, overlap   */
    CASTLING_ERR_UNSUPPORTED = -2, /* d not a multiple of 16 or > 128, ksize > 7, bad dtype  */
    CASTLING_ERR_ALIGNMENT = -3,   /* a tensor pointer is not 16-byte aligned                */
    CASTLING_ERR_ARCH = -4,        /* current device is not compute capability 10.x          */
    CASTLING_ERR_CUDA = -5,        /* a CUDA call failed; see castling_attn_last_cuda_error  */
    CASTLING_ERR_OOM = -6,         /* workspace allocation failed or exceeds max_workspace   */
    CASTLING_ERR_DEVICE = -7,      /* a kernel reported a bounded wait that ran out          */
    CASTLING_ERR_SCRATCH_LIMIT = -8 /* problem needs more than the built-in static scratch    */
};

/* Kernel families the dispatcher can be pinned to (testing and benchmarking). */
enum {
    CASTLING_PATH_AUTO = 0,
    CASTLING_PATH_SIMT = 1,   /* CUDA-core FMA kernels: every dtype, d and ksize supported   */
    CASTLING_PATH_TENSOR = 2  /* tcgen05/TMEM + TMA kernels: bf16, ksize 3 or 5, d = 64, or   */
                              /* d = 32 packed two tokens or two heads to a 128-byte row      */
};

typedef struct {
    int ksize;            /* depthwise filter side: odd, 1..7                                  */
    double eps;           /* floor on ||q||, ||k||; <= 0 selects the default 1e-12.  A zero    */
                          /* row therefore has cosine 0 with everything (similarity 1/2).     */
    int force_path;       /* CASTLING_PATH_*; AUTO picks by dtype, d and N                     */
    size_t max_workspace; /* cap on handle-owned device memory in bytes; 0 = no cap            */
    int prefix_tokens;    /* 0..16 leading tokens per sequence that have no grid position (class */
                          /* / distillation tokens).  N becomes prefix_tokens + gridH*gridW in     */
                          /* every forward call.  The paper does not say how such tokens meet the */
                          /* convolution; here they enter both attention terms of Eq. 9 like any  */
                          /* token (they add to K^^T V and to the token sum, and get an output    */
                          /* row), while DWConv and its bias act on the grid tokens only.         */
    /* Variants of the attention beyond the inference-time core; all zero selects the core.        */
    int normalize_rows;   /* 1: every row of attention weights is divided by its sum, the denominator */
                          /* of kernel-based linear attention (Sec. 3.1, Eq. 3) that Eq. 9 leaves out: */
                          /* the attention term of token t is divided by N/2 + q^_t . (sum_j k^_j)/pi; */
                          /* the convolution is added unchanged.  bf16 shapes that the tensor-core    */
                          /* kernels take run there; the rest on the CUDA-core kernels.               */
    int exact_kernel;     /* 1: the exact angular kernel 1 - arccos(q^.k^)/pi (Eq. 4-5) instead of its  */
                          /* kept part 1/2 + q^.k^/pi (Eq. 8).  Quadratic in N (explicit weights).     */
                          /* This flag and sparse_branch run on the tensor cores for bf16 heads of     */
                          /* width 64 (without normalize_rows and leading tokens), else on CUDA cores. */
    int sparse_branch;    /* 1: the auxiliary branch of training (Sec. 3.2.2, Eq. 10) is added to the   */
                          /* weights: Mask_eps(Softmax_j(q^_t . k^_j)), Mask_eps(p) = p if p > eps else */
                          /* 0; softmax over the keys of a query on the cosines of the unit rows, no    */
                          /* 1/sqrt(d), survivors not renormalised.  Quadratic in N.  The comparison    */
                          /* p > eps is taken in fp32.                                                 */
    double sparse_eps;    /* the mask's threshold (the paper uses 0.02 for classification)             */
} castling_attn_config_t;

/*
 * castling_attn_create: make a handle bound to the CURRENT CUDA device.
 *   cfg         host pointer, read once; NULL selects {ksize 3, eps 1e-12, AUTO, no cap, no prefix, no variant}.
 *               exact_kernel and sparse_branch take the explicit-weights kernel (any dtype and d, O(N^2 d)
 *               time, at most 16384 tokens, no prefix tokens, contiguous or strided device tensors).
 *   out_handle  host pointer receiving the handle; set to NULL on failure.
 * Allocates nothing on the device.  Errors: INVALID_ARG, UNSUPPORTED (ksize), ARCH, CUDA.
 */
CASTLING_API int castling_attn_create(const castling_attn_config_t* cfg, castling_attn_t** out_handle);

/*
 * castling_attn_forward: enqueue one forward pass on `stream` and return without
 * synchronising (Eq. 8-9 as stated at the top of this file).
 *
 *   q, k, v     DEVICE pointers, [B, H, N, d] contiguous, d innermost, N = prefix_tokens +
 *               gridH*gridW, grid token (y, x) at t = prefix_tokens + y*gridW + x.  Read only.
 *               16-byte aligned.
 *   dw_weight   DEVICE pointer, [H*d, ksize, ksize], same dtype as q.  Read only.
 *   dw_bias     DEVICE pointer, [H*d], same dtype, or NULL for no bias.
 *   out         DEVICE pointer, [B, H, N, d], same dtype; every element is written exactly
 *               once.  Must not overlap any input.  16-byte aligned.
 *   B,H,gridH,gridW,d   positive; d a multiple of 16, d <= 128.
 *   dtype       element type of all six tensors.
 *   stream      a cudaStream_t passed as void* (NULL = the legacy default stream).
 *
 * Ownership: the caller owns every tensor; the handle owns a workspace (partial and final
 * d x d states, token sums) that may be (re)allocated with cudaMalloc on the first call
 * for a larger shape -- that call synchronises the device; later calls of the same or a
 * smaller shape allocate nothing.
 * Such later calls only enqueue kernels on `stream` (no allocation, no synchronisation, no
 * host-side dependence on device results), so they can be recorded by stream capture and replayed
 * as a CUDA graph on new data in the same buffers.
 * A handle serves one host thread and one stream at a time; distinct handles are
 * independent.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, OOM, CUDA.  Nothing aborts
 * and no exception crosses this boundary.
 */
CASTLING_API int castling_attn_forward(castling_attn_t* handle,
                          const void* q, const void* k, const void* v,
                          const void* dw_weight, const void* dw_bias, void* out,
                          int B, int H, int gridH, int gridW, int d,
                          castling_dtype_t dtype, void* stream);

/*
 * Element strides of q, k, v and out for castling_attn_forward_strided.  Element (b, h, n, j)
 * of a tensor sits at  base + b*batch + h*head + n*token + j  (the d elements of a token are
 * always contiguous).  [B,H,N,d] contiguous is {H*N*d, N*d, d}; token-major [B,N,H,d], which is what a
 * projection layer produces without a transpose, is {N*H*d, d, H*d}; q taken out of a fused
 * [B,N,3,H,d] projection is {N*3*H*d, d, 3*H*d} with base = qkv + 0, H*d or 2*H*d.
 */
typedef struct {
    long long q_batch, q_head, q_token;
    long long k_batch, k_head, k_token;
    long long v_batch, v_head, v_token;
    long long out_batch, out_head, out_token;
} castling_attn_layout_t;

/*
 * castling_attn_forward_strided: castling_attn_forward for tensors that are not [B,H,N,d]
 * contiguous (same Eq. 8-9 computation; the paper does not prescribe a memory layout).
 *
 *   layout      HOST pointer, read during the call.  Every stride is in elements, >= 0, a multiple of
 *               16 bytes; token strides are >= d; batch (head) strides are > 0 when B (H) > 1.
 *   q,k,v,out   DEVICE base pointers (element (0,0,0,0)), 16-byte aligned.  The ranges spanned by
 *               `out` and by each input must not overlap, and distinct (b,h,n) of `out` must not
 *               share memory (not checked).
 *   everything else as for castling_attn_forward.
 *
 * The tensor-core kernels read such layouts directly through strided TMA descriptors: width-64
 * heads with any strides; width-32 heads when a 128-byte row holds either two adjacent tokens of one
 * head (contiguous tokens, even gridW and N) or the same token of two adjacent heads (head stride 32,
 * even H, as in token-major [B,N,H,32]).  Everything else, and any layout a descriptor cannot express,
 * runs on the CUDA-core kernels.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, OOM, CUDA.
 */
CASTLING_API int castling_attn_forward_strided(castling_attn_t* handle,
                          const void* q, const void* k, const void* v,
                          const void* dw_weight, const void* dw_bias, void* out,
                          int B, int H, int gridH, int gridW, int d,
                          castling_dtype_t dtype, const castling_attn_layout_t* layout, void* stream);

/*
 * castling_attn_forward_host: the same computation with every tensor in HOST memory.
 * Copies q, k, v, dw_weight and dw_bias to handle-owned device staging buffers on
 * `stream`, runs the forward pass, copies `out` back and synchronises the stream
 * before returning, so on return `out` holds the result.  Large problems are cut into chunks
 * of whole (b,h) planes whose uploads, kernels and downloads overlap on two internal copy streams
 * (created on first use); that needs pinned host memory to be effective, pageable memory also
 * works.  Because a chunk is a smaller problem, its token splits and hence the fp32 summation
 * order may differ from one castling_attn_forward call on the whole batch (same tolerance).  Shapes, dtype and
 * errors as for castling_attn_forward (alignment is not required of host pointers).
 */
CASTLING_API int castling_attn_forward_host(castling_attn_t* handle,
                               const void* q, const void* k, const void* v,
                               const void* dw_weight, const void* dw_bias, void* out,
                               int B, int H, int gridH, int gridW, int d,
                               castling_dtype_t dtype, void* stream);

/*
 * castling_attn_destroy: free the workspace and the handle.  The caller must have
 * synchronised every stream the handle was used on.  NULL is accepted.
 */
CASTLING_API int castling_attn_destroy(castling_attn_t* handle);

/* Bytes of handle-owned device workspace a forward of this shape needs (0 on bad arguments).  The
 * figure is for sequences of gridH*gridW tokens; a handle with prefix_tokens may need one more
 * partial-state slot per (b,h). */
CASTLING_API size_t castling_attn_workspace_bytes(int B, int H, int gridH, int gridW, int d, castling_dtype_t dtype);

/* Static, NUL-terminated description of a return code. */
CASTLING_API const char* castling_attn_error_string(int code);

/* The cudaError_t (as int) behind the handle's most recent CASTLING_ERR_CUDA / OOM, else 0. */
CASTLING_API int castling_attn_last_cuda_error(const castling_attn_t* handle);

/*
 * castling_attn_last_path: which kernel family (CASTLING_PATH_SIMT / _TENSOR) the handle's
 * most recent successful forward used, and how many kernels it launched (may be NULL).
 */
CASTLING_API int castling_attn_last_path(const castling_attn_t* handle, int* kernel_launches);

/*
 * castling_attn_device_status: read back the handle's device-side status word
 * (synchronises `stream`).  0 = every bounded wait in the kernels completed; otherwise
 * returns CASTLING_ERR_DEVICE and stores the raw word in *raw (may be NULL); a non-zero word is
 * reported once and cleared, together with the arrival counters a kernel may have left half way.
 */
CASTLING_API int castling_attn_device_status(castling_attn_t* handle, void* stream, unsigned int* raw);

/*
 * A forward whose token grid is cut into bands of rows held by different devices ("sequence sharding").  The
 * paper's complexity paragraph (Sec. 3.2.1) is what makes this cheap: everything the keys and values of the
 * whole sequence contribute to Eq. 9 is the d x d matrix K^^T V and the token sum of V, so the devices exchange
 * B*H*(d*d + d) floats, not tokens; the depthwise convolution needs the (ksize-1)/2 grid rows on either side
 * of a band from its neighbours.  The library does the two local halves; the caller sums the states over the
 * devices in between (one all-reduce) and supplies the neighbour rows of V.
 *
 * castling_attn_state_words(d) = d*d + d: floats per (b,h) of a state: S row-major [key feature][value
 * feature], then the token sum s.  Raw sums: the states of the bands of one sequence simply add up.
 *
 * castling_attn_shard_state: this band's sums.
 *   k, v        DEVICE, [B, H, n_tokens, d] contiguous: the band's tokens (their grid position does not matter).
 *   state_out   DEVICE, float [B*H][d*d + d], overwritten.
 * castling_attn_shard_apply: the band's output rows from a state summed over all bands.
 *   q, out      DEVICE, [B, H, gridH_local*gridW, d] contiguous: the band's queries / outputs.
 *   v_halo      DEVICE, [B, H, (halo_top + gridH_local + halo_bottom)*gridW, d]: the band's rows of V preceded by
 *               the last halo_top rows of the band above and followed by the first halo_bottom rows of the band
 *               below; each of the two is 0 at the edge of the whole grid (zero padding applies there) and at
 *               most (ksize-1)/2, and must be (ksize-1)/2 wherever a neighbouring band exists.
 *   state       DEVICE, float [B*H][d*d + d]: the sum over all bands of what castling_attn_shard_state wrote.
 * Both enqueue on `stream` and return (the first call of a larger shape may allocate the workspace).  bf16 bands of
 * width-64 heads with at least 48 tokens run on the tensor-core kernels (unless the handle is pinned to
 * CASTLING_PATH_SIMT), everything else on the CUDA-core kernels.  A handle created with prefix tokens or any variant flag:
 * UNSUPPORTED.  Pointers 16-byte aligned.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, OOM, CUDA.
 */
CASTLING_API size_t castling_attn_state_words(int d);
CASTLING_API int castling_attn_shard_state(castling_attn_t* handle, const void* k, const void* v, float* state_out,
                          int B, int H, int n_tokens, int d, castling_dtype_t dtype, void* stream);
CASTLING_API int castling_attn_shard_apply(castling_attn_t* handle, const void* q, const void* v_halo,
                          const void* dw_weight, const void* dw_bias, const float* state, void* out,
                          int B, int H, int gridH_local, int gridW, int halo_top, int halo_bottom, int d,
                          castling_dtype_t dtype, void* stream);

/*
 * castling_attn_selftest_wait: check the mechanism behind that status word without any fault.  Launches one
 * small kernel on `stream` whose threads wait, with a limit of `limit_us` microseconds (1 .. 1 000 000), on a
 * shared-memory barrier that nothing completes -- the situation of a pipeline whose copy or partner never
 * arrives.  The wait must give up, raise a bit in the status word and let the kernel return; the call
 * synchronises `stream` and returns CASTLING_OK when the kernel ran to its end that way.  Afterwards
 * castling_attn_device_status reports CASTLING_ERR_DEVICE once (raw word 16) and clears the word; the handle
 * stays usable.  May allocate the workspace header on first use.  (The paper has no counterpart: this
 * verifies the failure behaviour of the kernels' bounded waits.)
 */
CASTLING_API int castling_attn_selftest_wait(castling_attn_t* handle, unsigned int limit_us, void* stream);

/*
 * castling_attn_set_profiling: with enable != 0 every later forward on this handle records a
 * CUDA event on its stream before its first kernel and after each kernel.  Off by default;
 * the events add a little latency between kernels, so time whole forwards with it off.
 */
CASTLING_API int castling_attn_set_profiling(castling_attn_t* handle, int enable);

/*
 * castling_attn_kernel_times: per-kernel durations of the handle's most recent forward.
 * Waits for that forward to finish, writes up to `capacity` durations in milliseconds to
 * ms[] (host) and, if names is not NULL, static kernel-name strings to names[]; returns the
 * number written (0 when profiling is off), or a negative error code.
 */
CASTLING_API int castling_attn_kernel_times(castling_attn_t* handle, float* ms, const char** names, int capacity);

/*
 * castling_attn_forward_static: the same forward pass for callers that cannot allocate device
 * memory -- code running inside a region where cudaMalloc is forbidden or would stall everything
 * (a latency-critical serving loop, a plug-in that is handed a fixed memory budget by its host
 * application, a process whose allocator owns the whole GPU).  It takes no handle and calls no
 * cudaMalloc, cudaFree or any other allocating routine.  (The paper has no counterpart to this
 * entry point; it exists only for such callers.)
 *
 * The d x d states that pass from the state kernel to the apply kernel are kept in a fixed
 * CASTLING_STATIC_SCRATCH_BYTES (4 MiB) array that is part of the library's device image: every
 * GPU on which the library is loaded holds that array until the process exits.  A problem fits
 * when B*H*(d*d + d)*4 bytes <= CASTLING_STATIC_SCRATCH_BYTES (e.g. d = 64: B*H <= 252;
 * d = 32: B*H <= 992); larger ones return CASTLING_ERR_SCRATCH_LIMIT and nothing is launched.
 * The CUDA-core kernels are used for every dtype.
 *
 * Arguments as for castling_attn_forward, with the handle's configuration passed directly:
 * ksize (odd, 1..7) and eps (<= 0 selects 1e-12).  Tensors are DEVICE pointers, 16-byte aligned;
 * the call only enqueues on `stream`.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) with
 * that device current; make that first call outside any stream capture.  All calls on a device
 * share the one array and it keeps the last call's contents: nothing in it needs clearing
 * between calls (every word that is read is first overwritten by the same call), but two calls
 * whose kernels overlap on the GPU -- different streams, or the same problem from two threads --
 * race on it.  Serialise them on one stream.
 */
#define CASTLING_STATIC_SCRATCH_BYTES (4u << 20)
CASTLING_API int castling_attn_forward_static(const void* q, const void* k, const void* v,
                                              const void* dw_weight, const void* dw_bias, void* out,
                                              int B, int H, int gridH, int gridW, int d,
                                              int ksize, double eps, castling_dtype_t dtype, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CASTLING_ATTN_H_ */

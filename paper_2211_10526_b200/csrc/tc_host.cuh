// Host-side interface of the tensor-core (tcgen05 + TMA) path.
#pragma once

#include "castling_internal.cuh"
#include <cuda.h>

namespace castling {
namespace tc {

// Arrival counters per (b,h): one per group of splits (at most 64 / 4 groups) and one for the groups.
constexpr int kCountersPerHead = 17;

bool make_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                          const uint64_t* strides, const uint32_t* box, bool swizzle128);

// Width-32 heads, two adjacent tokens of one head per 128-byte row: contiguous tokens, even grid width,
// an even number of tokens per plane.
inline bool token_pairs(const Problem& p) {
    return p.d == 32 && p.gridW % 2 == 0 && p.N % 2 == 0 && p.contiguous_tokens();
}

// True when the tensor-core kernels can take this problem (bf16; d = 64, or d = 32 with even gridW;
// 3x3 or 5x5 filters).
bool supports(const Problem& p);

// True when automatic dispatch should pick them (enough rows per (b,h) to fill their tiles).
bool preferred(const Problem& p);

// 128-byte rows per (b,h): N for d = 64, N / 2 for d = 32 (two tokens per row).
int rows_per_head(int N, int d);

// Words of one (b,h) state as the tensor-core kernels store it (always the 64-wide form): S, s, and with row-sum
// normalisation the sum of the unit key rows behind them.
constexpr int kStateWords = 64 * 64 + 64;
constexpr int kStateWordsRownorm = kStateWords + 64;
inline int state_words_of(const Problem& p) { return p.rownorm ? kStateWordsRownorm : kStateWords; }

// Token splits of the tensor-core state kernel and the workspace words it needs beyond the state.
int choose_splits(int BH, int N);

// Enqueue state build, split reduction and apply for one problem.  `status` is the device status
// word; `counters` holds kCountersPerHead zero-initialised arrival counters per (b,h), left at zero by every call.  Returns the cudaError_t of the launches; cudaErrorNotSupported if a tensor map could not
// be built.
cudaError_t forward(const Problem& p, float* ws_state, float* ws_partial, unsigned* counters, int P,
                    unsigned* status, cudaStream_t stream, int* launches, KernelTimer* timer);

// The two halves of a forward on their own (a sequence sharded over devices): the state of a shard's tokens, written
// to state_out in the documented layout (S row-major, then s), and the apply pass over a band of grid rows with a
// state summed over all shards.  Head width 64 only (the width-32 packings keep their states in another form).
bool shard_supports(const Problem& p);
cudaError_t shard_state(const Problem& p, float* state_out, float* ws_partial, unsigned* counters, unsigned* status,
                        cudaStream_t stream, int* launches, KernelTimer* timer);
cudaError_t shard_apply(const Problem& p, const float* state, unsigned* status, cudaStream_t stream, int* launches,
                        KernelTimer* timer);

// Launchers of the individual kernels (each in its own file).
cudaError_t launch_state(const Problem& p, float* partial, float* final_state, unsigned* counters, int P,
                         int tiles_per_cta, unsigned* status, cudaStream_t st);
cudaError_t launch_apply(const Problem& p, const float* partial, int P, unsigned* status, cudaStream_t st);
// Output rows of the off-grid leading tokens (p.prefix of them per plane), from the final state.
cudaError_t launch_prefix_rows(const Problem& p, const float* state, cudaStream_t st);

// One-kernel forward (csrc/tc_pipe.cu): a state pipeline and an apply pipeline share every CTA; work is handed
// out, and progress is signalled, through counters in global memory.
// Counter layout: kPipeCtrHeader words (CTAs that have left, next patch to hand out, next chunk of rows to hand
// out, CTAs that have cleared their part of the states), then kPipeCtrPerPlane words per plane: chunks whose
// sums are added to the plane's state, patches applied, the plane's operand block is ready.  All zero between calls.
constexpr int kPipeCtrHeader = 4, kPipeCtrPerPlane = 4;
constexpr int kPipeCtrNextPatch = 1, kPipeCtrNextChunk = 2, kPipeCtrCleared = 3;
constexpr int kPipeCtrWritten = 0, kPipeCtrApplied = 1, kPipeCtrReady = 2;
struct PipePlan {
    bool ok;           // the one-kernel forward takes this shape
    int grid;          // CTAs (at most one per multiprocessor)
    int s_tiles;       // 64-row state tiles per plane
    int chunk_tiles;   // tiles per chunk of rows
    int n_chunks;      // chunks per plane
    int ahead;         // planes the state pipeline may run ahead of the apply pipeline
};
// rows: 128-byte rows per plane (leading tokens included); cols x gridH: the token grid in 128-byte columns.
PipePlan plan_pipe(int BH, int rows, int cols, int gridH);
bool pipe_supports(const Problem& p);
// The plane sums end up at state[plane] (cleared by the kernel itself); `ready` holds pipe_ready_words(BH) words
// for the per-plane operand blocks that the apply pipelines copy; ctr as described above.
size_t pipe_ready_words(int BH);
cudaError_t launch_pipe(const Problem& p, float* state, float* ready, unsigned* ctr, unsigned* status, cudaStream_t st);

// Forward with one thread-block cluster per plane (csrc/tc_cluster.cu): every CTA builds the state of its share of
// the plane, the cluster adds the shares up through distributed shared memory, every CTA applies the sum to its
// share of the patches.  One launch, no workspace.  cluster_size: CTAs per plane, 0 when the shape is not taken.
int cluster_size(const Problem& p);
cudaError_t launch_cluster(const Problem& p, int C, unsigned* status, cudaStream_t st);

// Single-kernel forward for short sequences (bf16, 3x3 or 5x5 filters, at most 256 128-byte rows per plane:
// d = 64 with N <= 256, two width-32 heads per row with N <= 256, or width-32 token pairs with N <= 512): no workspace.
bool fused_supports(const Problem& p);
cudaError_t launch_fused(const Problem& p, unsigned* status, cudaStream_t st);

// Attention with the exact angular kernel on the tensor cores (csrc/tc_quad.cu): explicit weights, bf16, head width 64.
bool quad_supports(const Problem& p);
cudaError_t launch_quad(const Problem& p, unsigned* status, cudaStream_t st);

// A one-CTA kernel whose bounded wait (limit_ns) can never be satisfied: it has to raise kStatusSelfTestTimeout in
// *status and return; *reached_end becomes 1 (2 if the wait claimed success).
cudaError_t launch_selftest_wait(unsigned* status, unsigned long long limit_ns, unsigned* reached_end, cudaStream_t st);

}  // namespace tc

// Shared with the CUDA-core path: sums P partial states per (b,h) in index order.
cudaError_t launch_reduce(const float* partial, float* state, int BH, int words, int P, cudaStream_t st);

}  // namespace castling

// Orchestration of the tensor-core path: state build -> split reduction -> apply, in stream order
// (the stream is the only synchronisation between the phases; no kernel waits on another).
#include "tc_host.cuh"

namespace castling {
namespace tc {

namespace {
constexpr int kStateTile = 128;  // tokens per UMMA stage of the state kernel
}

// bf16 with head width 64, or head width 32 on a grid of even width (two tokens share one
// 128-byte row there); 3x3 or 5x5 filters.
bool supports(const Problem& p) {
    if (!p.bf16 || (p.ksize != 3 && p.ksize != 5)) return false;
    // width-32 heads pair two adjacent tokens in one 128-byte row: the tokens must be contiguous
    return p.d == 64 || (p.d == 32 && p.gridW % 2 == 0 && p.contiguous_tokens());
}

int rows_per_head(int N, int d) { return d == 32 ? N / 2 : N; }

// With fewer than 48 rows per (b,h) the 128-row tiles of the tensor-core kernels are mostly padding
// and the CUDA-core kernels are faster (measured: 4x4 grids of width-32 heads, 20 us against 33 us).
bool preferred(const Problem& p) { return supports(p) && rows_per_head(p.N, p.d) >= 48; }

// Two state CTAs fit on an SM: as many splits as keep all CTAs of the launch resident at once
// (2 x 148), every split non-empty, at most 64 splits.
int choose_splits(int BH, int N) {
    const int tiles = (N + kStateTile - 1) / kStateTile;
    if (tiles < 1) return 1;
    int P = (2 * 148) / BH;
    if (P > tiles) P = tiles;
    if (P > 64) P = 64;
    if (P < 1) P = 1;
    const int per = (tiles + P - 1) / P;
    return (tiles + per - 1) / per;
}

cudaError_t forward(const Problem& p, float* ws_state, float* ws_partial, unsigned* counters, int P,
                    unsigned* status, cudaStream_t stream, int* launches, KernelTimer* timer) {
    *launches = 0;
    if (fused_supports(p)) {  // a whole (b,h) fits in shared memory: one kernel, no workspace
        const cudaError_t e = launch_fused(p, status, stream);
        if (e != cudaSuccess) return e;
        ++*launches;
        timer->mark(stream, "tc_fused");
        return cudaSuccess;
    }
    const int tiles = (rows_per_head(p.N, p.d) + kStateTile - 1) / kStateTile;
    const int per = (tiles + P - 1) / P;
    cudaError_t e = launch_state(p, ws_partial, ws_state, counters, P, per, status, stream);
    if (e != cudaSuccess) return e;
    ++*launches;
    timer->mark(stream, "tc_state");
    e = launch_apply(p, ws_state, 1, status, stream);
    if (e != cudaSuccess) return e;
    ++*launches;
    timer->mark(stream, "tc_apply");
    return cudaSuccess;
}

}  // namespace tc
}  // namespace castling

// Orchestration of the tensor-core path: state build -> split reduction -> apply, in stream order
// (the stream is the only synchronisation between the phases; no kernel waits on another).
#include "tc_host.cuh"

namespace castling {
namespace tc {

namespace {
constexpr int kStateTile = 128;  // tokens per UMMA stage of the state kernel
}

bool supports(const Problem& p) {
    return p.bf16 && p.d == 64 && (p.ksize == 3 || p.ksize == 5);
}

// Two state CTAs fit on an SM: as many splits as keep all CTAs of the launch resident at once
// (2 x 148), every split non-empty, at most 64 splits.
int choose_splits(int BH, int N) {
    const int tiles = (N + kStateTile - 1) / kStateTile;
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
    const int tiles = (p.N + kStateTile - 1) / kStateTile;
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

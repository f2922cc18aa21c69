// Orchestration of the tensor-core path: state build -> split reduction -> apply, in stream order
// (the stream is the only synchronisation between the phases; no kernel waits on another).
#include "tc_host.cuh"

#include <cstdlib>

namespace castling {
namespace tc {

namespace {
constexpr int kStateTile = 128;  // tokens per UMMA stage of the state kernel
}

namespace {
// Width-32 heads fill a 128-byte row in one of two ways: two adjacent tokens of one head (tokens
// contiguous, even grid width), or the same token of two adjacent heads (head stride 32, as in a
// token-major [B,N,H,32] tensor with an even number of heads).
bool head_pairs(const Problem& p) {
    return p.d == 32 && p.H % 2 == 0 && p.hdiv == p.H && p.head0 == 0 && p.lq.head == 32 && p.lk.head == 32 &&
           p.lv.head == 32 && p.lo.head == 32;
}
}  // namespace

// bf16, 3x3 or 5x5 filters, head width 64 or one of the two width-32 arrangements above.
bool supports(const Problem& p) {
    if (!p.bf16 || (p.ksize != 3 && p.ksize != 5)) return false;
    return p.d == 64 || token_pairs(p) || head_pairs(p);
}

int rows_per_head(int N, int d) { return d == 32 ? N / 2 : N; }

// With fewer than 48 rows per (b,h) the 128-row tiles of the tensor-core kernels are mostly padding
// and the CUDA-core kernels are faster (measured: 4x4 grids of width-32 heads, 20 us against 33 us).
bool preferred(const Problem& p) {
    if (!supports(p)) return false;
    const int rows = (p.d == 32 && !token_pairs(p)) ? p.N : rows_per_head(p.N, p.d);
    return rows >= 48;
}

// Two state CTAs fit on an SM: as many splits as keep all CTAs of the launch resident at once
// (two per multiprocessor), every split non-empty, at most 64 splits.
int choose_splits(int BH, int N) {
    const int tiles = (N + kStateTile - 1) / kStateTile;
    if (tiles < 1) return 1;
    int P = (2 * device_sm_count()) / BH;
    if (P > tiles) P = tiles;
    if (P > 64) P = 64;
    if (P < 1) P = 1;
    const int per = (tiles + P - 1) / P;
    return (tiles + per - 1) / per;
}

// CASTLING_TC_ONE_KERNEL=1 in the environment selects the one-kernel forward (state and apply pipelines side
// by side in every CTA) instead of the separate state and apply kernels, which measure faster (read once).
static bool two_kernels() {
    static const bool one = [] { const char* e = getenv("CASTLING_TC_ONE_KERNEL"); return e && e[0] == '1'; }();
    return !one;
}

// CASTLING_TC_CLUSTER=1 in the environment selects the cluster-per-plane forward where the shape allows it.
static bool cluster_enabled() {
    static const bool on = [] { const char* e = getenv("CASTLING_TC_CLUSTER"); return e && e[0] == '1'; }();
    return on;
}

cudaError_t forward(const Problem& p_in, float* ws_state, float* ws_partial, unsigned* counters, int P,
                    unsigned* status, cudaStream_t stream, int* launches, KernelTimer* timer) {
    *launches = 0;
    Problem p = p_in;
    if (p.d == 32 && !token_pairs(p)) {
        // heads (2m, 2m+1) side by side = one width-64 plane whose state is block diagonal
        p.d = 64; p.H /= 2; p.BH /= 2; p.hdiv = p.H; p.blockdiag = true;
        p.lq.head = p.lk.head = p.lv.head = p.lo.head = 64;
        P = choose_splits(p.BH, p.N);
    }
    if (!p.rownorm && fused_supports(p)) {  // a whole (b,h) fits in shared memory: one kernel, no workspace
        const cudaError_t e = launch_fused(p, status, stream);
        if (e != cudaSuccess) return e;
        ++*launches;
        timer->mark(stream, "tc_fused");
        return cudaSuccess;
    }
    cudaError_t e;
    if (const int C = (cluster_enabled() && !p.rownorm) ? cluster_size(p) : 0) {
        e = launch_cluster(p, C, status, stream);
        if (e != cudaSuccess) return e;
        ++*launches;
        timer->mark(stream, "tc_cluster");
        return cudaSuccess;
    }
    if (!two_kernels() && !p.rownorm && pipe_supports(p)) {
        // state and apply pipelines in one persistent kernel: V is read from memory once
        e = launch_pipe(p, ws_state, ws_partial, counters, status, stream);
        if (e != cudaSuccess) return e;
        ++*launches;
        timer->mark(stream, "tc_pipe");
    } else {
        const int tiles = (rows_per_head(p.N, p.d) + kStateTile - 1) / kStateTile;
        const int per = (tiles + P - 1) / P;
        e = launch_state(p, ws_partial, ws_state, counters, P, per, status, stream);
        if (e != cudaSuccess) return e;
        ++*launches;
        timer->mark(stream, "tc_state");
        e = launch_apply(p, ws_state, 1, status, stream);
        if (e != cudaSuccess) return e;
        ++*launches;
        timer->mark(stream, "tc_apply");
    }
    if (p.prefix > 0) {
        e = launch_prefix_rows(p, ws_state, stream);
        if (e != cudaSuccess) return e;
        ++*launches;
        timer->mark(stream, "tc_prefix_rows");
    }
    return cudaSuccess;
}

bool shard_supports(const Problem& p) {
    return p.bf16 && p.d == 64 && (p.ksize == 3 || p.ksize == 5) && p.prefix == 0 && !p.rownorm && p.N >= 48;
}

cudaError_t shard_state(const Problem& p, float* state_out, float* ws_partial, unsigned* counters, unsigned* status,
                        cudaStream_t stream, int* launches, KernelTimer* timer) {
    *launches = 0;
    const int P = choose_splits(p.BH, p.N);
    const int tiles = (p.N + kStateTile - 1) / kStateTile;
    const cudaError_t e = launch_state(p, ws_partial, state_out, counters, P, (tiles + P - 1) / P, status, stream);
    if (e != cudaSuccess) return e;
    ++*launches;
    timer->mark(stream, "tc_state");
    return cudaSuccess;
}

cudaError_t shard_apply(const Problem& p, const float* state, unsigned* status, cudaStream_t stream, int* launches,
                        KernelTimer* timer) {
    *launches = 0;
    const cudaError_t e = launch_apply(p, state, 1, status, stream);
    if (e != cudaSuccess) return e;
    ++*launches;
    timer->mark(stream, "tc_apply");
    return cudaSuccess;
}

}  // namespace tc
}  // namespace castling

// Attention with the explicit weights, one row of the N x N weight matrix at a time (CUDA cores, fp32
// arithmetic, any supported dtype): the variants of the method that have no form linear in N.
//     weights(t, j) = base(x) [/ sum_j base(x)] [+ Mask_eps(Softmax_j(x))],   x = q^_t . k^_j
//     base(x) = 1/2 + x/pi            the kept part of Eq. 8 (what the linear kernels compute re-associated)
//             = 1 - arccos(x)/pi      the exact angular kernel, Eq. 4-5
//     row-sum division: Eq. 3's denominator;  masked softmax: the auxiliary branch of training, Eq. 10,
//     Mask_eps(p) = p if p > eps else 0, softmax over the keys of one query, no 1/sqrt(d)
//     out_t = sum_j weights(t, j) v_j + bias + DWConv(V)_t                                   (Eq. 9)
// One CTA owns 64 queries of one (b,h) and walks over the keys in tiles of 64: unit rows of Q and K in
// shared memory, a 64 x 64 tile of cosines per step on a 4 x 4 register block per thread, the weights of
// the tile in shared memory, then the 64 x d product with the V tile.  The softmax denominators need all
// keys, so the masked branch takes a first sweep over the keys for them.  O(N^2 d) time, O(N d) memory.
#include "castling_internal.cuh"

#include <math_constants.h>

namespace castling {
namespace {

constexpr int kThreads = 256;
constexpr int kTile = 64;   // queries per CTA, keys per step

template <typename T> struct Io;
template <> struct Io<float> {
    static __device__ __forceinline__ float load(const float* p) { return __ldg(p); }
    static __device__ __forceinline__ void store(float* p, float x) { *p = x; }
};
template <> struct Io<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16* p) {
        return __uint_as_float(((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};

// `rows` token rows of width D, starting `first` tokens into the plane, as fp32 into a tile with row stride LD;
// rows at or beyond `valid` are zero.  With `unit` every row is divided by max(||row||, eps).
template <typename T, int D, int LD>
__device__ __forceinline__ void stage_tile(const T* __restrict__ plane, long long tok, int first, int valid,
                                           float* __restrict__ s, bool unit, float eps2) {
    for (int c = threadIdx.x; c < kTile * D; c += kThreads) {
        const int r = c / D, i = c % D;
        s[r * LD + i] = (r < valid) ? Io<T>::load(plane + (long long)(first + r) * tok + i) : 0.f;
    }
    __syncthreads();
    if (unit) {
        // four threads per row
        const int r = threadIdx.x >> 2, l = threadIdx.x & 3;
        float ss = 0.f;
        for (int i = l; i < D; i += 4) { const float x = s[r * LD + i]; ss = fmaf(x, x, ss); }
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        ss += __shfl_xor_sync(0xffffffffu, ss, 2);
        const float rn = 1.0f / sqrtf(fmaxf(ss, eps2));
        for (int i = l; i < D; i += 4) s[r * LD + i] *= rn;
        __syncthreads();
    }
}

struct QuadParams {
    int H, head0, hdiv, gridH, gridW, ksize, N;
    int exact;          // 1: exact angular kernel, 0: its kept linear part
    int rownorm;        // divide every row of base weights by its sum
    int sparse;         // add the masked softmax
    float sparse_eps, eps2;
    Layout lq, lk, lv, lo;
};

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
quad_attention_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                      const T* __restrict__ w, const T* __restrict__ bias, T* __restrict__ out, const QuadParams prm) {
    constexpr int LD = D + 1;          // Q and K tiles: conflict-free column walks
    constexpr int LP = kTile + 1;      // weight tile
    constexpr int R = D / 16;          // channels per thread in the product with V
    extern __shared__ __align__(16) float smem[];
    float* qs = smem;                      // [64][D+1] unit rows of the queries
    float* ks = qs + kTile * LD;           // [64][D+1] unit rows of the keys of this step
    float* vs = ks + kTile * LD;           // [64][D]   values of this step
    float* ps = vs + kTile * D;            // [64][65]  weights of this step

    const int N = prm.N, tiles = (N + kTile - 1) / kTile;
    const int bh = blockIdx.x / tiles, t0 = (blockIdx.x % tiles) * kTile;
    const int q_valid = min(kTile, N - t0);
    const T* qb = q + plane_offset(prm.lq, bh, prm.hdiv);
    const T* kb = k + plane_offset(prm.lk, bh, prm.hdiv);
    const T* vb = v + plane_offset(prm.lv, bh, prm.hdiv);
    T* ob = out + plane_offset(prm.lo, bh, prm.hdiv);

    stage_tile<T, D, LD>(qb, prm.lq.token, t0, q_valid, qs, true, prm.eps2);

    const int tq = threadIdx.x / 16, tk = threadIdx.x % 16;   // cosine block: queries tq + 16 r, keys tk + 16 c
    const int tj = tk;                                         // product with V: channels tj * R ..

    // cosines of this thread's 4 x 4 block against the key tile in ks
    auto cosines = [&](float (&x)[4][4]) {
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) x[r][c] = 0.f;
#pragma unroll 4
        for (int i = 0; i < D; ++i) {
            float a[4], b[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) a[r] = qs[(tq + 16 * r) * LD + i];
#pragma unroll
            for (int c = 0; c < 4; ++c) b[c] = ks[(tk + 16 * c) * LD + i];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) x[r][c] = fmaf(a[r], b[c], x[r][c]);
        }
    };
    // sum over the 16 threads that share a query (lanes tk of a half warp)
    auto row_sum = [](float x) {
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        return x;
    };

    float zinv[4] = {0.f, 0.f, 0.f, 0.f};
    if (prm.sparse) {
        // first sweep: softmax denominators sum_j exp(x_tj) (cosines lie in [-1, 1]: no running maximum needed)
        float z[4] = {0.f, 0.f, 0.f, 0.f};
        for (int j0 = 0; j0 < N; j0 += kTile) {
            const int k_valid = min(kTile, N - j0);
            __syncthreads();
            stage_tile<T, D, LD>(kb, prm.lk.token, j0, k_valid, ks, true, prm.eps2);
            float x[4][4];
            cosines(x);
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                float part = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) part += (tk + 16 * c < k_valid) ? expf(x[r][c]) : 0.f;
                z[r] += row_sum(part);
            }
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) zinv[r] = 1.0f / z[r];
    }

    // acc_b: base weights times V (divided by the row sum at the end when asked); acc_s: masked softmax times V
    float acc_b[4][R], acc_s[4][R];
    float den[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < R; ++c) { acc_b[r][c] = 0.f; acc_s[r][c] = 0.f; }
    // acc[r][c] += sum_j ps[query tq + 16 r][j] * vs[j][channel tj * R + c]
    auto times_v = [&](float (&acc)[4][R]) {
#pragma unroll 4
        for (int j = 0; j < kTile; ++j) {
            float a[4], b[R];
#pragma unroll
            for (int r = 0; r < 4; ++r) a[r] = ps[(tq + 16 * r) * LP + j];
#pragma unroll
            for (int c = 0; c < R; ++c) b[c] = vs[j * D + tj * R + c];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < R; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
        }
    };

    for (int j0 = 0; j0 < N; j0 += kTile) {
        const int k_valid = min(kTile, N - j0);
        __syncthreads();   // the previous step's tiles are consumed
        for (int c = threadIdx.x; c < kTile * D; c += kThreads) {
            const int r = c / D, i = c % D;
            vs[c] = (r < k_valid) ? Io<T>::load(vb + (long long)(j0 + r) * prm.lv.token + i) : 0.f;
        }
        stage_tile<T, D, LD>(kb, prm.lk.token, j0, k_valid, ks, true, prm.eps2);
        float x[4][4];
        cosines(x);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            float part = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float xc = fminf(1.0f, fmaxf(-1.0f, x[r][c]));  // rounding may leave [-1, 1]
                float base = prm.exact ? 1.0f - acosf(xc) * (1.0f / CUDART_PI_F) : fmaf(x[r][c], kInvPi, 0.5f);
                if (tk + 16 * c >= k_valid) base = 0.f;
                part += base;
                ps[(tq + 16 * r) * LP + tk + 16 * c] = base;
            }
            den[r] += row_sum(part);
        }
        __syncthreads();
        times_v(acc_b);
        if (prm.sparse) {
            __syncthreads();
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float p = expf(x[r][c]) * zinv[r];
                    ps[(tq + 16 * r) * LP + tk + 16 * c] = (tk + 16 * c < k_valid && p > prm.sparse_eps) ? p : 0.f;
                }
            __syncthreads();
            times_v(acc_s);
        }
    }

    // out = [base part / row sum] + sparse part + bias + depthwise convolution of V on the grid
    const int h = (prm.head0 + bh) % prm.H;
    const int KK = prm.ksize * prm.ksize, rad = (prm.ksize - 1) / 2;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int tl = tq + 16 * r;
        if (tl >= q_valid) continue;
        const int t = t0 + tl, y = t / prm.gridW, xg = t % prm.gridW;
        const float scale = prm.rownorm ? 1.0f / den[r] : 1.0f;
        float o[R];
#pragma unroll
        for (int c = 0; c < R; ++c) {
            const int ch = h * D + tj * R + c;
            o[c] = fmaf(acc_b[r][c], scale, acc_s[r][c]) + (bias ? Io<T>::load(bias + ch) : 0.f);
        }
        for (int dy = -rad; dy <= rad; ++dy) {
            const int yy = y + dy;
            if (yy < 0 || yy >= prm.gridH) continue;
            for (int dx = -rad; dx <= rad; ++dx) {
                const int xx = xg + dx;
                if (xx < 0 || xx >= prm.gridW) continue;
                const T* vp = vb + (long long)(yy * prm.gridW + xx) * prm.lv.token + tj * R;
#pragma unroll
                for (int c = 0; c < R; ++c) {
                    const int ch = h * D + tj * R + c;
                    o[c] = fmaf(Io<T>::load(w + (size_t)ch * KK + (dy + rad) * prm.ksize + (dx + rad)), Io<T>::load(vp + c), o[c]);
                }
            }
        }
#pragma unroll
        for (int c = 0; c < R; ++c) Io<T>::store(ob + (long long)t * prm.lo.token + tj * R + c, o[c]);
    }
}

template <int D> constexpr size_t quad_smem() {
    return sizeof(float) * ((size_t)2 * kTile * (D + 1) + (size_t)kTile * D + (size_t)kTile * (kTile + 1));
}

template <typename T, int D>
cudaError_t launch_quad(const Problem& p, cudaStream_t st) {
    QuadParams prm;
    prm.H = p.H; prm.head0 = p.head0; prm.hdiv = p.hdiv; prm.gridH = p.gridH; prm.gridW = p.gridW;
    prm.ksize = p.ksize; prm.N = p.N;
    prm.exact = p.exact_kernel ? 1 : 0; prm.rownorm = p.rownorm ? 1 : 0; prm.sparse = p.sparse ? 1 : 0;
    prm.sparse_eps = p.sparse_eps; prm.eps2 = p.eps2;
    prm.lq = p.lq; prm.lk = p.lk; prm.lv = p.lv; prm.lo = p.lo;
    constexpr size_t smem = quad_smem<D>();
    static PerDevice opt_in;
    if (smem > 48 * 1024) {
        const cudaError_t e = opt_in_smem(quad_attention_kernel<T, D>, smem, opt_in);
        if (e != cudaSuccess) return e;
    }
    const int tiles = (p.N + kTile - 1) / kTile;
    quad_attention_kernel<T, D><<<(unsigned)(p.BH * tiles), kThreads, smem, st>>>(
        static_cast<const T*>(p.q), static_cast<const T*>(p.k), static_cast<const T*>(p.v), static_cast<const T*>(p.w),
        static_cast<const T*>(p.bias), static_cast<T*>(p.out), prm);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_quad_d(const Problem& p, cudaStream_t st) {
    switch (p.d) {
        case 16: return launch_quad<T, 16>(p, st);
        case 32: return launch_quad<T, 32>(p, st);
        case 48: return launch_quad<T, 48>(p, st);
        case 64: return launch_quad<T, 64>(p, st);
        case 80: return launch_quad<T, 80>(p, st);
        case 96: return launch_quad<T, 96>(p, st);
        case 112: return launch_quad<T, 112>(p, st);
        case 128: return launch_quad<T, 128>(p, st);
        default: return cudaErrorNotSupported;
    }
}

}  // namespace

// The explicit-weights forward for one validated problem (no leading tokens).
cudaError_t quad_forward(const Problem& p, cudaStream_t stream, int* launches, KernelTimer* timer) {
    const cudaError_t e = p.bf16 ? launch_quad_d<__nv_bfloat16>(p, stream) : launch_quad_d<float>(p, stream);
    if (e != cudaSuccess) return e;
    *launches = 1;
    timer->mark(stream, "quad_attention");
    return cudaSuccess;
}

}  // namespace castling

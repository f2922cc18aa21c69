// CUDA-core (FMA) kernels of the linear-angular attention core.
//
// These cover every supported dtype, head width and filter size; the fp32 I/O
// path always runs here because its 1e-5 tolerance rules out bf16 operands.
//
//   state kernel  : per (b,h) and token split, k^ = k / max(||k||, eps),
//                   S += k^^T v (d x d), s += v           (Eq. 9, K^T V and the 1/2 term)
//   reduce kernel : sums the token splits in a fixed order (only when P > 1)
//   apply kernel  : out_t = (1/pi) q^_t S + 1/2 s + bias + DWConv(V)_t    (Eq. 9)
//   fused kernel  : all three steps in one CTA per (b,h) when a whole plane (at most 256 tokens)
//                   fits in shared memory: one launch, no workspace
#include "castling_internal.cuh"
#include "tc_host.cuh"

namespace castling {
namespace {

constexpr int kThreads = 256;
constexpr int kStateTile = 32;  // tokens staged per step of the state kernel
constexpr int kApplyTile = 64;  // tokens per CTA of the apply kernel

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kVec = 4;  // elements per 16-byte load
    static __device__ __forceinline__ void load16(const float* p, float (&f)[4]) {
        const float4 x = __ldg(reinterpret_cast<const float4*>(p));
        f[0] = x.x; f[1] = x.y; f[2] = x.z; f[3] = x.w;
    }
    static __device__ __forceinline__ float load1(const float* p) { return __ldg(p); }
    static __device__ __forceinline__ void store1(float* p, float x) { *p = x; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    static __device__ __forceinline__ void load16(const __nv_bfloat16* p, float (&f)[8]) {
        const uint4 x = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16* p) {
        return __uint_as_float(((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
    static __device__ __forceinline__ void store1(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};

// Copy `rows` token rows of width D (row r starts r * tok elements after g) into a padded fp32
// shared tile; rows at or beyond `valid` are zero-filled.
template <typename T, int D, int LD>
__device__ __forceinline__ void stage_rows(const T* __restrict__ g, long long tok, float* __restrict__ s, int rows, int valid) {
    constexpr int V = Elem<T>::kVec;
    constexpr int kChunksPerRow = D / V;
    for (int c = threadIdx.x; c < rows * kChunksPerRow; c += kThreads) {
        const int r = c / kChunksPerRow, col = (c % kChunksPerRow) * V;
        float f[V];
        if (r < valid) {
            Elem<T>::load16(g + r * tok + col, f);
        } else {
#pragma unroll
            for (int i = 0; i < V; ++i) f[i] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < V; ++i) s[r * LD + col + i] = f[i];
    }
}

// The same copy for a whole plane of `rows` valid rows, four 16-byte loads in flight per thread.
template <typename T, int D, int LD>
__device__ __forceinline__ void stage_plane(const T* __restrict__ g, long long tok, float* __restrict__ s, int rows) {
    constexpr int V = Elem<T>::kVec;
    constexpr int kChunksPerRow = D / V;
    constexpr int U = 4;
    const int total = rows * kChunksPerRow;
    for (int c0 = threadIdx.x; c0 < total; c0 += U * kThreads) {
        float f[U][V];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + u * kThreads;
            if (c < total) Elem<T>::load16(g + (c / kChunksPerRow) * tok + (c % kChunksPerRow) * V, f[u]);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = c0 + u * kThreads;
            if (c < total) {
                const int r = c / kChunksPerRow, col = (c % kChunksPerRow) * V;
#pragma unroll
                for (int i = 0; i < V; i += 4)
                    *reinterpret_cast<float4*>(s + r * LD + col + i) = make_float4(f[u][i], f[u][i + 1], f[u][i + 2], f[u][i + 3]);
            }
        }
    }
}

// 1 / max(||row||, eps) for ROWS rows of a shared tile, kThreads / ROWS lanes per row.
template <int D, int LD, int ROWS>
__device__ __forceinline__ void row_rnorm(const float* __restrict__ s, float* __restrict__ rn, float eps2) {
    constexpr int L = kThreads / ROWS;  // lanes per row: 8 (state) or 4 (apply)
    const int r = threadIdx.x / L, l = threadIdx.x % L;
    float ss = 0.f;
    for (int i = l; i < D; i += L) { const float x = s[r * LD + i]; ss = fmaf(x, x, ss); }
#pragma unroll
    for (int o = L / 2; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (l == 0) rn[r] = 1.0f / sqrtf(fmaxf(ss, eps2));
}

// ---------------------------------------------------------------------------
// state kernel: grid (BH * P).  CTA bh * P + p covers tokens [p*chunk, min(N,(p+1)*chunk)).
// Writes raw sums [S (d*d, row i = key feature, col j = value feature) | s (d)], `words` apart per split;
// with zsum the sum of the unit key rows (d words) follows: the row-sum denominator of Eq. 3 needs it.
// Thread (ti, tj) of a 16 x 16 arrangement owns an R x R block of S, R = D / 16.
// ---------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
simt_state_kernel(const T* __restrict__ k, const T* __restrict__ v, float* __restrict__ dst,
                  int N, int chunk, int P, float eps2, Layout lk, Layout lv, int hdiv, int words, int zsum) {
    constexpr int R = D / 16;
    constexpr int LD = D + 4;  // padded row, keeps 16-byte alignment
    __shared__ __align__(16) float ks[kStateTile * LD];
    __shared__ __align__(16) float vs[kStateTile * LD];
    __shared__ float rk[kStateTile];

    const int p = blockIdx.x % P, bh = blockIdx.x / P;
    const int n_begin = p * chunk, n_end = min(N, n_begin + chunk);
    const T* kb = k + plane_offset(lk, bh, hdiv);
    const T* vb = v + plane_offset(lv, bh, hdiv);
    const int ti = threadIdx.x / 16, tj = threadIdx.x % 16;

    float acc[R][R];
    float vsum[R], ksum[R];
#pragma unroll
    for (int a = 0; a < R; ++a) {
        vsum[a] = 0.f; ksum[a] = 0.f;
#pragma unroll
        for (int b = 0; b < R; ++b) acc[a][b] = 0.f;
    }

    for (int n0 = n_begin; n0 < n_end; n0 += kStateTile) {
        const int valid = min(kStateTile, n_end - n0);
        __syncthreads();  // previous tile fully consumed
        stage_rows<T, D, LD>(kb + n0 * lk.token, lk.token, ks, kStateTile, valid);
        stage_rows<T, D, LD>(vb + n0 * lv.token, lv.token, vs, kStateTile, valid);
        __syncthreads();
        row_rnorm<D, LD, kStateTile>(ks, rk, eps2);
        __syncthreads();
#pragma unroll 4
        for (int n = 0; n < kStateTile; ++n) {
            const float r = rk[n];
            float a[R], b[R];
#pragma unroll
            for (int x = 0; x < R; ++x) { a[x] = ks[n * LD + ti * R + x] * r; b[x] = vs[n * LD + tj * R + x]; }
#pragma unroll
            for (int x = 0; x < R; ++x) {
                vsum[x] += b[x];
                ksum[x] += a[x];
#pragma unroll
                for (int y = 0; y < R; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
            }
        }
    }

    float* out = dst + ((size_t)bh * P + p) * words;
#pragma unroll
    for (int x = 0; x < R; ++x)
#pragma unroll
        for (int y = 0; y < R; ++y) out[(ti * R + x) * D + tj * R + y] = acc[x][y];
    if (ti == 0) {
#pragma unroll
        for (int y = 0; y < R; ++y) out[D * D + tj * R + y] = vsum[y];
    }
    if (zsum && tj == 0) {
#pragma unroll
        for (int x = 0; x < R; ++x) out[D * D + D + ti * R + x] = ksum[x];
    }
}

// reduce kernel: grid (BH), sums P partial states in index order (bitwise reproducible).
__global__ void __launch_bounds__(kThreads)
simt_reduce_kernel(const float* __restrict__ partial, float* __restrict__ state, int words, int P) {
    const float* src = partial + (size_t)blockIdx.x * P * words;
    float* dst = state + (size_t)blockIdx.x * words;
    for (int i = threadIdx.x; i < words; i += kThreads) {
        float s = 0.f;
        for (int p = 0; p < P; ++p) s += src[(size_t)p * words + i];
        dst[i] = s;
    }
}

// ---------------------------------------------------------------------------
// apply kernel: grid (BH * ceil(N / 64)).  Each CTA produces 64 consecutive tokens of one
// (b,h): (1/pi) q^ S + 1/2 s + bias + depthwise conv of V (zero padding), one store each.
// Thread (tq, tj) owns tokens tq + 16 r (r = 0..3) and channels tj*R .. tj*R + R - 1.
// ---------------------------------------------------------------------------
template <int D> constexpr size_t simt_apply_smem(int ksize) {
    return sizeof(float) * ((size_t)D * D + 3 * D + (size_t)ksize * ksize * D + kApplyTile * (D + 1) + 2 * kApplyTile);
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
simt_apply_kernel(const T* __restrict__ q, const T* __restrict__ v, const T* __restrict__ w,
                  const T* __restrict__ bias, const float* __restrict__ state, T* __restrict__ out,
                  int H, int head0, int prefix, int gridH, int gridW, int ksize, float eps2, Layout lq, Layout lv,
                  Layout lo, int hdiv, int words, int zsum, int v_row0, int v_rows) {
    // v_row0, v_rows: the V tensor holds v_rows grid rows, of which row v_row0 is this call's grid row 0 (a shard of
    // a taller grid brings the rows of its neighbours that the filters reach; otherwise 0 and gridH)
    constexpr int R = D / 16;
    constexpr int LDQ = D + 1;
    extern __shared__ __align__(16) float smem[];
    const int KK = ksize * ksize, rad = (ksize - 1) / 2;
    float* S_sm = smem;                 // [D][D], scaled by 1/pi
    float* c_sm = S_sm + D * D;         // [D]    1/2 s
    float* b_sm = c_sm + D;             // [D]    bias of the convolution (grid tokens only)
    float* w_sm = b_sm + D;             // [KK][D] filters of this head, tap-major
    float* qs = w_sm + KK * D;          // [64][D+1]
    float* rq = qs + kApplyTile * LDQ;  // [64]
    float* rden = rq + kApplyTile;      // [64] 1 / (row sum of the similarities), or 1
    float* z_sm = rden + kApplyTile;    // [D]  sum of the unit key rows (zsum only)

    const int N = prefix + gridH * gridW;
    const int tiles = (N + kApplyTile - 1) / kApplyTile;
    const int bh = blockIdx.x / tiles, h = (head0 + bh) % H;
    const int t0 = (blockIdx.x % tiles) * kApplyTile;
    const int valid = min(kApplyTile, N - t0);
    const float* st = state + (size_t)bh * words;

    for (int i = threadIdx.x; i < D * D; i += kThreads) S_sm[i] = st[i] * kInvPi;
    for (int i = threadIdx.x; i < D; i += kThreads) {
        c_sm[i] = 0.5f * st[D * D + i];
        z_sm[i] = zsum ? st[D * D + D + i] : 0.f;
        b_sm[i] = bias ? Elem<T>::load1(bias + h * D + i) : 0.f;
    }
    for (int i = threadIdx.x; i < KK * D; i += kThreads) {
        const int tap = i / D, ch = i % D;
        w_sm[i] = Elem<T>::load1(w + ((size_t)(h * D + ch)) * KK + tap);
    }
    {   // Q tile; rows are padded by one float, so staged with scalar stores
        constexpr int V = Elem<T>::kVec;
        const T* qb = q + plane_offset(lq, bh, hdiv) + t0 * lq.token;
        for (int c = threadIdx.x; c < kApplyTile * (D / V); c += kThreads) {
            const int r = c / (D / V), col = (c % (D / V)) * V;
            float f[V];
            if (r < valid) {
                Elem<T>::load16(qb + r * lq.token + col, f);
            } else {
#pragma unroll
                for (int i = 0; i < V; ++i) f[i] = 0.f;
            }
#pragma unroll
            for (int i = 0; i < V; ++i) qs[r * LDQ + col + i] = f[i];
        }
    }
    __syncthreads();
    row_rnorm<D, LDQ, kApplyTile>(qs, rq, eps2);
    __syncthreads();
    if (threadIdx.x < kApplyTile) {
        // Eq. 3's denominator for the kept kernel of Eq. 8: sum_j (1/2 + q^.k^_j/pi) = N/2 + q^ . (sum_j k^_j)/pi
        float den = 1.0f;
        if (zsum) {
            float dot = 0.f;
            for (int i = 0; i < D; ++i) dot = fmaf(qs[threadIdx.x * LDQ + i], z_sm[i], dot);
            den = fmaf(dot * rq[threadIdx.x], kInvPi, 0.5f * (float)N);
        }
        rden[threadIdx.x] = 1.0f / den;
    }
    __syncthreads();

    const int tq = threadIdx.x / 16, tj = threadIdx.x % 16;
    float acc[4][R];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < R; ++c) acc[r][c] = 0.f;

#pragma unroll 4
    for (int i = 0; i < D; ++i) {
        float a[4], b[R];
#pragma unroll
        for (int r = 0; r < 4; ++r) a[r] = qs[(tq + 16 * r) * LDQ + i];
#pragma unroll
        for (int c = 0; c < R; ++c) b[c] = S_sm[i * D + tj * R + c];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < R; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
    }

    const T* vb = v + plane_offset(lv, bh, hdiv);
    T* ob = out + plane_offset(lo, bh, hdiv);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int tl = tq + 16 * r;
        if (tl >= valid) continue;
        const int t = t0 + tl, g = t - prefix, y = g / gridW, x = g % gridW;  // g < 0: an off-grid leading token
        const float scale = rq[tl], inv_rowsum = rden[tl];
        float o[R];
#pragma unroll
        for (int c = 0; c < R; ++c) {
            // without the denominator: one rounding fewer, as before
            o[c] = zsum ? fmaf(acc[r][c], scale, c_sm[tj * R + c]) * inv_rowsum + (g >= 0 ? b_sm[tj * R + c] : 0.f)
                        : fmaf(acc[r][c], scale, c_sm[tj * R + c] + (g >= 0 ? b_sm[tj * R + c] : 0.f));
        }
        for (int dy = -rad; dy <= rad && g >= 0; ++dy) {
            const int yy = y + dy + v_row0;
            if (yy < 0 || yy >= v_rows) continue;
            for (int dx = -rad; dx <= rad; ++dx) {
                const int xx = x + dx;
                if (xx < 0 || xx >= gridW) continue;
                const T* vp = vb + (prefix + yy * gridW + xx) * lv.token + tj * R;
                const float* wp = w_sm + ((dy + rad) * ksize + (dx + rad)) * D + tj * R;
#pragma unroll
                for (int c = 0; c < R; ++c) o[c] = fmaf(wp[c], Elem<T>::load1(vp + c), o[c]);
            }
        }
#pragma unroll
        for (int c = 0; c < R; ++c) Elem<T>::store1(ob + t * lo.token + tj * R + c, o[c]);
    }
}

// ---------------------------------------------------------------------------
// fused kernel for short sequences: grid (BH), one CTA per (b,h).  K, V and Q of the plane sit in
// shared memory as fp32 for the whole pass, so the state never leaves the SM, V is read from
// memory once for both the state and the convolution, and the forward is a single launch with
// no workspace.  The arithmetic order per element is that of the three-kernel path with P = 1.
// ---------------------------------------------------------------------------
// It is taken when at least two such CTAs fit on an SM and there are enough planes to occupy the
// device (measured: 64 x 8 planes of 7 x 7 tokens 22.7 -> 17.8 us, 64 x 12 of 4 x 4 20.6 -> 15.1 us;
// 8 planes of 14 x 14 are faster on the three-kernel path, which spreads a plane over several CTAs).
constexpr int kFusedMaxTokens = 256;
constexpr int kFusedMinPlanes = 64;
constexpr size_t kFusedSmemLimit = 100 * 1024;

template <int D> constexpr size_t simt_fused_smem(int N, int ksize) {
    return sizeof(float) * (3 * (size_t)N * (D + 4) + 2 * (size_t)N + (size_t)D * D + 2 * D + (size_t)ksize * ksize * D);
}

// 1 / max(||row||, eps) for `rows` rows of a shared tile, one warp per row at a time.
template <int D, int LD>
__device__ __forceinline__ void row_rnorm_warp(const float* __restrict__ s, float* __restrict__ rn, int rows, float eps2) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r < rows; r += kThreads / 32) {
        float ss = 0.f;
        for (int i = lane; i < D; i += 32) { const float x = s[r * LD + i]; ss = fmaf(x, x, ss); }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) rn[r] = 1.0f / sqrtf(fmaxf(ss, eps2));
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
simt_fused_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                  const T* __restrict__ w, const T* __restrict__ bias, T* __restrict__ out,
                  int H, int head0, int prefix, int gridH, int gridW, int ksize, float eps2, Layout lq, Layout lk,
                  Layout lv, Layout lo, int hdiv) {
    constexpr int R = D / 16;
    constexpr int LD = D + 4;
    extern __shared__ __align__(16) float smem[];
    const int N = prefix + gridH * gridW;
    const int KK = ksize * ksize, rad = (ksize - 1) / 2;
    float* ks = smem;               // [N][LD]
    float* vs = ks + N * LD;        // [N][LD]
    float* qs = vs + N * LD;        // [N][LD]
    float* rk = qs + N * LD;        // [N]
    float* rq = rk + N;             // [N]
    float* S_sm = rq + N;           // [D][D], scaled by 1/pi
    float* c_sm = S_sm + D * D;     // [D]    1/2 s
    float* b_sm = c_sm + D;         // [D]    bias of the convolution (grid tokens only)
    float* w_sm = b_sm + D;         // [KK][D] filters of this head, tap-major

    const int bh = blockIdx.x, h = (head0 + bh) % H;
    stage_plane<T, D, LD>(k + plane_offset(lk, bh, hdiv), lk.token, ks, N);
    stage_plane<T, D, LD>(v + plane_offset(lv, bh, hdiv), lv.token, vs, N);
    stage_plane<T, D, LD>(q + plane_offset(lq, bh, hdiv), lq.token, qs, N);
    for (int i = threadIdx.x; i < KK * D; i += kThreads) {
        const int tap = i / D, ch = i % D;
        w_sm[i] = Elem<T>::load1(w + ((size_t)(h * D + ch)) * KK + tap);
    }
    __syncthreads();
    row_rnorm_warp<D, LD>(ks, rk, N, eps2);
    row_rnorm_warp<D, LD>(qs, rq, N, eps2);
    __syncthreads();

    const int ti = threadIdx.x / 16, tj = threadIdx.x % 16;
    {   // state: thread (ti, tj) owns an R x R block of S
        float acc[R][R];
        float vsum[R];
#pragma unroll
        for (int a = 0; a < R; ++a) {
            vsum[a] = 0.f;
#pragma unroll
            for (int b = 0; b < R; ++b) acc[a][b] = 0.f;
        }
#pragma unroll 4
        for (int n = 0; n < N; ++n) {
            const float r = rk[n];
            float a[R], b[R];
#pragma unroll
            for (int x = 0; x < R; ++x) { a[x] = ks[n * LD + ti * R + x] * r; b[x] = vs[n * LD + tj * R + x]; }
#pragma unroll
            for (int x = 0; x < R; ++x) {
                vsum[x] += b[x];
#pragma unroll
                for (int y = 0; y < R; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
            }
        }
#pragma unroll
        for (int x = 0; x < R; ++x)
#pragma unroll
            for (int y = 0; y < R; ++y) S_sm[(ti * R + x) * D + tj * R + y] = acc[x][y] * kInvPi;
        if (ti == 0) {
#pragma unroll
            for (int y = 0; y < R; ++y) {
                const int ch = tj * R + y;
                c_sm[ch] = 0.5f * vsum[y];
                b_sm[ch] = bias ? Elem<T>::load1(bias + h * D + ch) : 0.f;
            }
        }
    }
    __syncthreads();

    // apply: thread (tq, tj) owns tokens t0 + tq + 16 r (r = 0..3) and channels tj*R .. tj*R + R - 1
    const int tq = ti;
    T* ob = out + plane_offset(lo, bh, hdiv);
    for (int t0 = 0; t0 < N; t0 += kApplyTile) {
        float acc[4][R];
        int row[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            row[r] = min(t0 + tq + 16 * r, N - 1);  // clamped rows are computed and dropped
#pragma unroll
            for (int c = 0; c < R; ++c) acc[r][c] = 0.f;
        }
#pragma unroll 4
        for (int i = 0; i < D; ++i) {
            float a[4], b[R];
#pragma unroll
            for (int r = 0; r < 4; ++r) a[r] = qs[row[r] * LD + i];
#pragma unroll
            for (int c = 0; c < R; ++c) b[c] = S_sm[i * D + tj * R + c];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < R; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int t = t0 + tq + 16 * r;
            if (t >= N) continue;
            const int g = t - prefix, y = g / gridW, x = g % gridW;  // g < 0: an off-grid leading token
            const float scale = rq[t];
            float o[R];
#pragma unroll
            for (int c = 0; c < R; ++c) o[c] = fmaf(acc[r][c], scale, c_sm[tj * R + c] + (g >= 0 ? b_sm[tj * R + c] : 0.f));
            for (int dy = -rad; dy <= rad && g >= 0; ++dy) {
                const int yy = y + dy;
                if (yy < 0 || yy >= gridH) continue;
                for (int dx = -rad; dx <= rad; ++dx) {
                    const int xx = x + dx;
                    if (xx < 0 || xx >= gridW) continue;
                    const float* vp = vs + (prefix + yy * gridW + xx) * LD + tj * R;
                    const float* wp = w_sm + ((dy + rad) * ksize + (dx + rad)) * D + tj * R;
#pragma unroll
                    for (int c = 0; c < R; ++c) o[c] = fmaf(wp[c], vp[c], o[c]);
                }
            }
#pragma unroll
            for (int c = 0; c < R; ++c) Elem<T>::store1(ob + t * lo.token + tj * R + c, o[c]);
        }
    }
}

template <typename T, int D>
cudaError_t launch_simt(const Problem& p, float* ws_state, float* ws_partial, int P,
                        cudaStream_t stream, int* launches, KernelTimer* timer) {
    const int zsum = p.rownorm ? 1 : 0;
    const int words = D * D + D + (zsum ? D : 0);
    if (!zsum && p.phase == kPhaseAll && p.N <= kFusedMaxTokens && p.BH >= kFusedMinPlanes &&
        simt_fused_smem<D>(p.N, p.ksize) <= kFusedSmemLimit) {
        const size_t smem = simt_fused_smem<D>(p.N, p.ksize);
        static PerDevice fused_opt_in;
        cudaError_t e = opt_in_smem(simt_fused_kernel<T, D>, kFusedSmemLimit, fused_opt_in);
        if (e != cudaSuccess) return e;
        simt_fused_kernel<T, D><<<(unsigned)p.BH, kThreads, smem, stream>>>(
            static_cast<const T*>(p.q), static_cast<const T*>(p.k), static_cast<const T*>(p.v),
            static_cast<const T*>(p.w), static_cast<const T*>(p.bias), static_cast<T*>(p.out),
            p.H, p.head0, p.prefix, p.gridH, p.gridW, p.ksize, p.eps2, p.lq, p.lk, p.lv, p.lo, p.hdiv);
        e = cudaGetLastError();
        if (e == cudaSuccess) *launches = 1;
        timer->mark(stream, "simt_fused");
        return e;
    }
    cudaError_t e = cudaSuccess;
    if (p.phase != kPhaseApplyOnly) {
        const int tiles = (p.N + kStateTile - 1) / kStateTile;
        const int chunk = ((tiles + P - 1) / P) * kStateTile;
        float* dst = (P > 1) ? ws_partial : ws_state;
        simt_state_kernel<T, D><<<(unsigned)(p.BH * P), kThreads, 0, stream>>>(
            static_cast<const T*>(p.k), static_cast<const T*>(p.v), dst, p.N, chunk, P, p.eps2, p.lk, p.lv, p.hdiv, words, zsum);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
        timer->mark(stream, "simt_state");
        if (P > 1) {
            simt_reduce_kernel<<<p.BH, kThreads, 0, stream>>>(ws_partial, ws_state, words, P);
            e = cudaGetLastError();
            if (e != cudaSuccess) return e;
            ++*launches;
            timer->mark(stream, "simt_reduce");
        }
        if (p.phase == kPhaseStateOnly) return cudaSuccess;
    }
    const size_t smem = simt_apply_smem<D>(p.ksize);
    static PerDevice apply_opt_in;
    e = opt_in_smem(simt_apply_kernel<T, D>, simt_apply_smem<D>(7), apply_opt_in);  // 7 x 7: the largest filter
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)(p.BH * ((p.N + kApplyTile - 1) / kApplyTile));
    simt_apply_kernel<T, D><<<grid, kThreads, smem, stream>>>(
        static_cast<const T*>(p.q), static_cast<const T*>(p.v), static_cast<const T*>(p.w),
        static_cast<const T*>(p.bias), ws_state, static_cast<T*>(p.out), p.H, p.head0, p.prefix, p.gridH, p.gridW, p.ksize,
        p.eps2, p.lq, p.lv, p.lo, p.hdiv, words, zsum, p.v_row0, p.v_rows > 0 ? p.v_rows : p.gridH);
    e = cudaGetLastError();
    if (e == cudaSuccess) ++*launches;
    timer->mark(stream, "simt_apply");
    return e;
}

template <int D>
cudaError_t launch_simt_dtype(const Problem& p, float* s, float* part, int P, cudaStream_t st, int* n,
                              KernelTimer* t) {
    return p.bf16 ? launch_simt<__nv_bfloat16, D>(p, s, part, P, st, n, t)
                  : launch_simt<float, D>(p, s, part, P, st, n, t);
}

}  // namespace

cudaError_t launch_reduce(const float* partial, float* state, int BH, int words, int P, cudaStream_t st) {
    simt_reduce_kernel<<<BH, kThreads, 0, st>>>(partial, state, words, P);
    return cudaGetLastError();
}

bool simt_supports(int d, int ksize) {
    return d >= 16 && d <= 128 && d % 16 == 0 && ksize >= 1 && ksize <= 7 && (ksize & 1);
}

// Token splits of the state kernel: enough CTAs to fill the device about twice over,
// at least four staged tiles per split, capped at 64.
int simt_choose_splits(int BH, int N) {
    const int tiles = (N + kStateTile - 1) / kStateTile;
    int P = (2 * device_sm_count() + BH - 1) / BH;
    if (P > tiles / 4) P = tiles / 4;
    if (P > 64) P = 64;
    if (P < 1) P = 1;
    return P;
}

cudaError_t simt_forward(const Problem& p, float* ws_state, float* ws_partial, int P,
                         cudaStream_t stream, int* launches, KernelTimer* timer) {
    *launches = 0;
    switch (p.d) {
        case 16: return launch_simt_dtype<16>(p, ws_state, ws_partial, P, stream, launches, timer);
        case 32: return launch_simt_dtype<32>(p, ws_state, ws_partial, P, stream, launches, timer);
        case 48: return launch_simt_dtype<48>(p, ws_state, ws_partial, P, stream, launches, timer);
        case 64: return launch_simt_dtype<64>(p, ws_state, ws_partial, P, stream, launches, timer);
        case 80: return launch_simt_dtype<80>(p, ws_state, ws_partial, P, stream, launches, timer);
        case 96: return launch_simt_dtype<96>(p, ws_state, ws_partial, P, stream, launches, timer);
        case 112: return launch_simt_dtype<112>(p, ws_state, ws_partial, P, stream, launches, timer);
        case 128: return launch_simt_dtype<128>(p, ws_state, ws_partial, P, stream, launches, timer);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace castling

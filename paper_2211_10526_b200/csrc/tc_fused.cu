// Whole forward pass in one kernel for short sequences (bf16, at most 256 128-byte rows per (b,h): head
// width 64, two width-32 heads side by side, or width-32 heads with two adjacent tokens per row):
//     out_t = (1/pi) q^_t (K^^T V) + 1/2 sum_n v_n + bias + DWConv(V)_t                    (Eq. 9)
// A plane (one (b,h)) fits in shared memory, so K, V and Q come from memory once, the state never
// leaves the SM and the forward is a single launch without workspace.  Two CTAs share an SM; each
// walks over planes blockIdx.x, blockIdx.x + gridDim.x, ...  Per plane
//   warp 0      TMA: K, V and Q as one or two 128-token tiles each (128-byte swizzle; rows beyond N
//               are zero-filled); once the state UMMAs have retired, V again without swizzle into
//               the K buffer (an L2 hit), which is what the convolution reads
//   warps 2..9  thread = token row: scale the K row by 1 / max(||k||, eps) in place; 1 / max(||q||, eps)
//   warp 1      one thread issues the state UMMAs, A = [K^ ; 1 0 0 ...] (M-major, the ones row makes
//               accumulator row 64 the token sum of V), B = V (N-major): S and s land in TMEM
//   warps 2..9  read S and s from TMEM, write S' = S / pi as the bf16 B operand of the second
//               contraction and s as fp32
//   warp 1      apply UMMAs: acc[tile] = Q[tile] * S' into TMEM (the state's columns are reused)
//   warps 2..9  thread = token: accumulator rows from TMEM to shared memory as fp32 (over the swizzled
//               V tile and the Q tile, both dead by then); then lane = channel pair, warp = a run of
//               eight tokens of one grid row: depthwise convolution with the filters in registers and a
//               sliding window along x, out = acc / max(||q||, eps) + 1/2 s + bias + conv, one rounding
//               to bf16, 128-byte rows stored straight to memory; leading off-grid tokens get the
//               attention terms only
#include "tc_common.cuh"
#include "tc_host.cuh"

namespace castling {
namespace tc {
namespace {

constexpr int kD = 64;
constexpr int kTile = 128;                       // tokens per UMMA tile
constexpr int kMaxTiles = 2;
constexpr int kTileBytes = kTile * kD * 2;       // 16 KiB
constexpr int kBufBytes = kMaxTiles * kTileBytes;
constexpr int kWorkers = 256;                    // warps 2..9
constexpr int kThreads = 64 + kWorkers;
constexpr int kTmemCols = 128;                   // [0,64): state, then tile 0 of the output; [64,128): tile 1
constexpr int kSeg = 8;                          // tokens of one grid row per convolution unit

// Shared memory: K | V | Q | S' | ones | rq | s | zeros | barriers.  After their first use the buffers change
// role: K holds the unswizzled V plane, V and Q hold the fp32 accumulator rows of tiles 0 and 1.
constexpr int kOffK = 0, kOffV = kBufBytes, kOffQ = 2 * kBufBytes;
constexpr int kOffS = 3 * kBufBytes;            // S' 64 x 64 bf16
constexpr int kOffOnes = kOffS + 8192;          // constant block of the A operand (after K: positive offset)
constexpr int kRqStride = 256 + kSeg;           // ragged units read up to kSeg - 1 entries past token N - 1
constexpr int kOffRq = kOffOnes + 2048;         // [2][kRqStride] 1 / max(||q||, eps); second row: second half (blockdiag)
constexpr int kOffSum = kOffRq + 2 * kRqStride * 4;  // [64] token sum of V
constexpr int kOffZero = kOffSum + kD * 4;      // 128 B of zeros: the convolution's padding
constexpr int kOffBar = kOffZero + 128;
constexpr size_t kSmemBytes = 1024 + kOffBar + 128;

struct FusedParams {
    const __nv_bfloat16* w;     // [H*64][KS][KS]
    const __nv_bfloat16* bias;  // [H*64] or nullptr
    __nv_bfloat16* out;         // token n of plane i at plane_offset(lo, i, hdiv) + n * lo.token
    Layout lo;
    int blockdiag;              // the plane is two width-32 heads side by side
    int H, head0, BH, hdiv, prefix, N, gridH, gridW;  // N = prefix + gridH * gridW
    float eps2;
    unsigned* status;
};

// OUT_PACKED: the output's token rows are contiguous (stride 64), which keeps the row addresses of the
// store loop compile-time offsets.
// TOKPAIR: width-32 heads with two adjacent tokens per 128-byte row (rows = N / 2): each half of a row has
// its own norm, the state is the sum of the two diagonal 32 x 32 blocks of the accumulator, used for both
// halves, and a lane of the convolution phase stands for (token parity, channel pair).
template <int KS, bool OUT_PACKED, bool TOKPAIR>
__global__ void __launch_bounds__(kThreads, (KS == 3) ? 2 : 1)
tc_fused_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmVplain,
                const FusedParams prm) {
    constexpr int R = KS / 2;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* K_s = smem + kOffK;
    uint8_t* V_s = smem + kOffV;
    uint8_t* Q_s = smem + kOffQ;
    uint8_t* S_s = smem + kOffS;
    uint8_t* ones = smem + kOffOnes;
    float* rq_s = reinterpret_cast<float*>(smem + kOffRq);
    float* sum_s = reinterpret_cast<float*>(smem + kOffSum);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kOffBar);
    uint64_t* k_full = bars + 0;      // TMA: K landed
    uint64_t* v_full = bars + 1;      // TMA: V (swizzled) landed
    uint64_t* q_full = bars + 2;      // TMA: Q landed
    uint64_t* vp_full = bars + 3;     // TMA: V (plain) landed in the K buffer
    uint64_t* k_scaled = bars + 4;    // K rows normalised (kWorkers)
    uint64_t* s_done = bars + 5;      // state UMMAs retired: S readable, K and V tiles no longer read
    uint64_t* sp_ready = bars + 6;    // S' and s written, state columns of TMEM read out (kWorkers)
    uint64_t* o_done = bars + 7;      // apply UMMAs retired: accumulators readable, Q tile no longer read
    uint64_t* tm_free = bars + 8;     // output accumulators read out of TMEM (kWorkers)
    uint64_t* plane_free = bars + 9;  // every buffer of the plane is free again (kWorkers)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int W = prm.gridW;
    const int N = TOKPAIR ? prm.N / 2 : prm.N;  // 128-byte rows per plane
    const bool halves = TOKPAIR || prm.blockdiag;  // each half of a row is normalised on its own
    const int tiles = (N + kTile - 1) / kTile;  // 1 or 2
    const int n_planes = (prm.BH - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    constexpr unsigned kBit = kStatusFusedTimeout;

    if (tid == 0) {
        mbar_init(k_full, 1); mbar_init(v_full, 1); mbar_init(q_full, 1); mbar_init(vp_full, 1);
        mbar_init(k_scaled, kWorkers); mbar_init(s_done, 1); mbar_init(sp_ready, kWorkers);
        mbar_init(o_done, 1); mbar_init(tm_free, kWorkers); mbar_init(plane_free, kWorkers);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmVplain);
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    if (warp >= 2 && tid - 64 < 128) {
        // constant block of A: for each of 16 token rows, element 64 (first of the second 64-wide
        // block along M) is 1.0 and the rest 0; 16-byte chunk c of row r sits at chunk c ^ (r & 7)
        const int t = tid - 64, r = t >> 3, c = t & 7;
        uint4 val = make_uint4(0, 0, 0, 0);
        if ((c ^ (r & 7)) == 0) val.x = 0x3f80u;
        *reinterpret_cast<uint4*>(ones + r * 128 + c * 16) = val;
        if (t < 8) *reinterpret_cast<uint4*>(smem + kOffZero + t * 16) = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t pol = l2_policy_evict_first();  // K and Q are read once
            int issued = 0, issued_vp = 0;
            for (int it = 0; it < n_planes; ++it) {
                const int bh = blockIdx.x + it * gridDim.x, pb = bh / prm.hdiv, ph = bh - pb * prm.hdiv;
                if (it > 0 && !mbar_wait(plane_free, (it - 1) & 1, abort_flag, prm.status, kBit)) break;
                mbar_expect_tx(k_full, tiles * kTileBytes);
                for (int t = 0; t < tiles; ++t) tma_load_4d_hint(K_s + t * kTileBytes, &tmK, k_full, 0, t * kTile, ph, pb, pol);
                mbar_expect_tx(v_full, tiles * kTileBytes);
                for (int t = 0; t < tiles; ++t) tma_load_4d(V_s + t * kTileBytes, &tmV, v_full, 0, t * kTile, ph, pb);
                mbar_expect_tx(q_full, tiles * kTileBytes);
                for (int t = 0; t < tiles; ++t) tma_load_4d_hint(Q_s + t * kTileBytes, &tmQ, q_full, 0, t * kTile, ph, pb, pol);
                ++issued;
                // the K tiles are dead once the state UMMAs have retired: bring V in again, unswizzled
                if (!mbar_wait(s_done, it & 1, abort_flag, prm.status, kBit)) break;
                mbar_expect_tx(vp_full, tiles * kTileBytes);
                for (int t = 0; t < tiles; ++t) tma_load_4d(K_s + t * kTileBytes, &tmVplain, vp_full, 0, t * kTile, ph, pb);
                ++issued_vp;
            }
            if (*abort_flag) {
                // giving up: let the copies in flight land before shared memory goes away
                if (issued) {
                    const uint32_t ph = (issued - 1) & 1;
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(k_full, ph); ++spin) {}
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(v_full, ph); ++spin) {}
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(q_full, ph); ++spin) {}
                }
                if (issued_vp) for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(vp_full, (issued_vp - 1) & 1); ++spin) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_state = umma_idesc_bf16(128, kD, true, true);
            constexpr uint32_t idesc_apply = umma_idesc_bf16(128, kD, false, true);
            const uint32_t k_addr = smem_u32(K_s), v_addr = smem_u32(V_s), q_addr = smem_u32(Q_s);
            const uint32_t s_addr = smem_u32(S_s), ones_addr = smem_u32(ones);
            for (int it = 0; it < n_planes; ++it) {
                const uint32_t ph = it & 1;
                if (!mbar_wait(k_scaled, ph, abort_flag, prm.status, kBit)) break;
                if (!mbar_wait(v_full, ph, abort_flag, prm.status, kBit)) break;
                // the previous plane's output accumulators share TMEM columns with this plane's state
                if (it > 0 && !mbar_wait(tm_free, (it - 1) & 1, abort_flag, prm.status, kBit)) break;
                tcgen05_fence_after_sync();
                for (int t = 0; t < tiles; ++t) {
#pragma unroll
                    for (int j = 0; j < kTile / 16; ++j) {  // one UMMA per 16 tokens (K = 16)
                        const uint32_t a0 = k_addr + t * kTileBytes + j * 2048, b0 = v_addr + t * kTileBytes + j * 2048;
                        umma_bf16(tmem, umma_desc_sw128(a0, ones_addr - a0, 1024), umma_desc_sw128(b0, 0, 1024),
                                  idesc_state, (t | j) != 0);
                    }
                }
                umma_commit(s_done);
                if (!mbar_wait(sp_ready, ph, abort_flag, prm.status, kBit)) break;
                if (!mbar_wait(q_full, ph, abort_flag, prm.status, kBit)) break;
                tcgen05_fence_after_sync();
                for (int t = 0; t < tiles; ++t) {
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k)
                        umma_bf16(tmem + t * kD, umma_desc_sw128(q_addr + t * kTileBytes + k * 32, 0, 1024),
                                  umma_desc_sw128(s_addr + k * 2048, 0, 1024), idesc_apply, k != 0);
                }
                umma_commit(o_done);
            }
        }
    } else {
        const int wt = tid - 64;                    // 0..255: the token row this thread normalises
        const int ww = warp - 2;                    // worker warp 0..7
        const int quarter = warp & 3;               // TMEM lanes 32*quarter .. +31 are this warp's
        const int half = ww >> 2;                   // thread = token phases: channels half*32 .. half*32 + 31
        const int r = quarter * 32 + lane;          // thread = token phases: row of both tiles
        const int Wc = TOKPAIR ? W / 2 : W;        // 128-byte columns per grid row
        const int segs = (Wc + kSeg - 1) / kSeg, n_units = prm.gridH * segs;
        const float2 zero2 = make_float2(0.f, 0.f);
        for (int it = 0; it < n_planes; ++it) {
            const uint32_t ph = it & 1;
            const int bh = blockIdx.x + it * gridDim.x;
            const int h = (prm.head0 + bh) % prm.H;
            // raw filter taps and bias of this lane's channel pair: loaded now, converted right before the
            // convolution, so that the round trip to L2 hides behind everything in between
            unsigned short wraw[2][KS * KS], braw[2] = {0, 0};
            {
                const int ch0 = TOKPAIR ? h * 32 + 2 * (lane & 15) : h * kD + 2 * lane;  // first channel of the lane's pair
                const unsigned short* w0 = reinterpret_cast<const unsigned short*>(prm.w) + (size_t)ch0 * (KS * KS);
#pragma unroll
                for (int i = 0; i < KS * KS; ++i) { wraw[0][i] = __ldg(w0 + i); wraw[1][i] = __ldg(w0 + KS * KS + i); }
                if (prm.bias) {
                    const unsigned short* b0 = reinterpret_cast<const unsigned short*>(prm.bias) + ch0;
                    braw[0] = __ldg(b0); braw[1] = __ldg(b0 + 1);
                }
            }
            // ---- K row -> unit row, in place ----
            if (!mbar_wait(k_full, ph, abort_flag, prm.status, kBit)) break;
            if (wt < N) {
                uint8_t* row = K_s + wt * 128;
                uint4 c[8];
                float2 ss[4] = {zero2, zero2, zero2, zero2};  // two chains for each half of the row
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    c[j] = *reinterpret_cast<const uint4*>(row + ((j ^ (wt & 7)) << 4));
                    const uint32_t w4[4] = {c[j].x, c[j].y, c[j].z, c[j].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 p = make_float2(bf16lo(w4[e]), bf16hi(w4[e]));
                        ss[2 * (j >> 2) + (e & 1)] = ffma2(p, p, ss[2 * (j >> 2) + (e & 1)]);
                    }
                }
                const float sa = (ss[0].x + ss[0].y) + (ss[1].x + ss[1].y), sb = (ss[2].x + ss[2].y) + (ss[3].x + ss[3].y);
                const float rka = 1.0f / sqrtf(fmaxf(halves ? sa : sa + sb, prm.eps2));
                const float rkb = halves ? 1.0f / sqrtf(fmaxf(sb, prm.eps2)) : rka;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t w4[4] = {c[j].x, c[j].y, c[j].z, c[j].w};
                    const float2 rk2 = (j < 4) ? make_float2(rka, rka) : make_float2(rkb, rkb);
                    uint32_t o4[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 p = ffma2(make_float2(bf16lo(w4[e]), bf16hi(w4[e])), rk2, zero2);
                        o4[e] = pack_bf16x2(p.x, p.y);
                    }
                    *reinterpret_cast<uint4*>(row + ((j ^ (wt & 7)) << 4)) = make_uint4(o4[0], o4[1], o4[2], o4[3]);
                }
                fence_proxy_async_smem();
            }
            mbar_arrive(k_scaled);

            // ---- 1 / max(||q||, eps) of row wt ----
            if (!mbar_wait(q_full, ph, abort_flag, prm.status, kBit)) break;
            if (wt < N) {
                const uint8_t* qrow = Q_s + wt * 128;
                float2 ss[4] = {zero2, zero2, zero2, zero2};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint4 c = *reinterpret_cast<const uint4*>(qrow + ((j ^ (wt & 7)) << 4));
                    const uint32_t w4[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 p = make_float2(bf16lo(w4[e]), bf16hi(w4[e]));
                        ss[2 * (j >> 2) + (e & 1)] = ffma2(p, p, ss[2 * (j >> 2) + (e & 1)]);
                    }
                }
                const float sa = (ss[0].x + ss[0].y) + (ss[1].x + ss[1].y), sb = (ss[2].x + ss[2].y) + (ss[3].x + ss[3].y);
                rq_s[wt] = rsqrtf(fmaxf(halves ? sa : sa + sb, prm.eps2));
                rq_s[kRqStride + wt] = rsqrtf(fmaxf(sb, prm.eps2));  // read only when the halves are separate heads
            }

            // ---- S, s out of TMEM -> S' (bf16 operand) and s ----
            if (!mbar_wait(s_done, ph, abort_flag, prm.status, kBit)) break;
            tcgen05_fence_after_sync();
            if (quarter < 3) {
                float a[32];
                {
                    float a0[16], a1[16];
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + half * 32, a0);
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + half * 32 + 16, a1);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e) { a[e] = a0[e]; a[16 + e] = a1[e]; }
                }
                if constexpr (TOKPAIR) {
                    // the two diagonal blocks meet in shared memory (the swizzled V tile is dead by now):
                    // [2][32 rows][32] fp32, 16-byte chunk c of row i at chunk c ^ (i & 7)
                    float* scr = reinterpret_cast<float*>(V_s) + quarter * 1024 + lane * 32;
                    if (quarter < 2 && quarter == half) {
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            *reinterpret_cast<float4*>(scr + ((e ^ (lane & 7)) << 2)) = make_float4(a[4 * e], a[4 * e + 1], a[4 * e + 2], a[4 * e + 3]);
                    }
                } else if (quarter < 2) {  // row r of S (key feature r), 32 value features
                    const float sp = (prm.blockdiag && quarter != half) ? 0.f : kInvPi;  // other head's block: zero
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint4 o;
                        o.x = pack_bf16x2(a[8 * e + 0] * sp, a[8 * e + 1] * sp);
                        o.y = pack_bf16x2(a[8 * e + 2] * sp, a[8 * e + 3] * sp);
                        o.z = pack_bf16x2(a[8 * e + 4] * sp, a[8 * e + 5] * sp);
                        o.w = pack_bf16x2(a[8 * e + 6] * sp, a[8 * e + 7] * sp);
                        *reinterpret_cast<uint4*>(S_s + r * 128 + (((half * 4 + e) ^ (r & 7)) << 4)) = o;
                    }
                }
                if (quarter == 2 && lane == 0) {  // accumulator row 64: the token sum of V
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        *reinterpret_cast<float4*>(sum_s + half * 32 + 4 * e) = make_float4(a[4 * e], a[4 * e + 1], a[4 * e + 2], a[4 * e + 3]);
                }
            }
            if constexpr (TOKPAIR) {
                named_barrier_sync(2, kWorkers);  // both diagonal blocks are in shared memory
                if (quarter < 2) {  // operand = blockdiag(S32, S32) / pi with S32 = block(0,0) + block(1,1)
                    const float* s0 = reinterpret_cast<const float*>(V_s) + lane * 32;
                    const float* s1 = s0 + 1024;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint4 o = make_uint4(0, 0, 0, 0);
                        if (quarter == half) {
                            const int c0 = ((2 * e) ^ (lane & 7)) << 2, c1 = ((2 * e + 1) ^ (lane & 7)) << 2;
                            const float4 x0 = *reinterpret_cast<const float4*>(s0 + c0), y0 = *reinterpret_cast<const float4*>(s1 + c0);
                            const float4 x1 = *reinterpret_cast<const float4*>(s0 + c1), y1 = *reinterpret_cast<const float4*>(s1 + c1);
                            o.x = pack_bf16x2((x0.x + y0.x) * kInvPi, (x0.y + y0.y) * kInvPi);
                            o.y = pack_bf16x2((x0.z + y0.z) * kInvPi, (x0.w + y0.w) * kInvPi);
                            o.z = pack_bf16x2((x1.x + y1.x) * kInvPi, (x1.y + y1.y) * kInvPi);
                            o.w = pack_bf16x2((x1.z + y1.z) * kInvPi, (x1.w + y1.w) * kInvPi);
                        }
                        *reinterpret_cast<uint4*>(S_s + r * 128 + (((half * 4 + e) ^ (r & 7)) << 4)) = o;
                    }
                }
            }
            fence_proxy_async_smem();
            tcgen05_fence_before_sync();
            mbar_arrive(sp_ready);

            // ---- accumulator rows out of TMEM -> fp32 rows in shared memory ----
            // Row r of tile t goes to the V buffer (t = 0) or the Q buffer (t = 1), 256 bytes per row,
            // 16-byte chunk c at chunk c ^ (r & 7): conflict-free for these row-per-thread writes and for
            // the row-per-warp reads below.  All UMMAs and all row-norm reads of those buffers are done:
            // o_done follows sp_ready, which every worker reaches after its reads of Q.
            if (!mbar_wait(o_done, ph, abort_flag, prm.status, kBit)) break;
            tcgen05_fence_after_sync();
#pragma unroll
            for (int t = 0; t < kMaxTiles; ++t) {
                if (t < tiles) {
                    uint8_t* srow = (t == 0 ? V_s : Q_s) + r * 256;
                    float a0[16], a1[16];
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + t * kD + half * 32, a0);
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + t * kD + half * 32 + 16, a1);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        *reinterpret_cast<float4*>(srow + (((half * 8 + e) ^ (r & 7)) << 4)) =
                            make_float4(a0[4 * e], a0[4 * e + 1], a0[4 * e + 2], a0[4 * e + 3]);
                        *reinterpret_cast<float4*>(srow + (((half * 8 + 4 + e) ^ (r & 7)) << 4)) =
                            make_float4(a1[4 * e], a1[4 * e + 1], a1[4 * e + 2], a1[4 * e + 3]);
                    }
                }
            }
            tcgen05_fence_before_sync();
            mbar_arrive(tm_free);
            if (!mbar_wait(vp_full, ph, abort_flag, prm.status, kBit)) break;
            named_barrier_sync(1, kWorkers);  // accumulator rows, rq and s are visible to every worker

            // ---- convolution + combine: lane = channel pair, warp = up to eight tokens of one grid row ----
            float2 wreg[KS][KS];
#pragma unroll
            for (int dy = 0; dy < KS; ++dy)
#pragma unroll
                for (int dx = 0; dx < KS; ++dx)
                    wreg[dy][dx] = make_float2(__uint_as_float((uint32_t)wraw[0][dy * KS + dx] << 16),
                                               __uint_as_float((uint32_t)wraw[1][dy * KS + dx] << 16));
            if constexpr (TOKPAIR) {
                // lane = (token parity, channel pair): a 128-byte row of the plain V plane, of the accumulator rows
                // and of the output holds tokens (2c, 2c+1) of a grid row; tokens are 64 bytes apart
                const int tp = lane >> 4, cp = lane & 15;
                const float2 hs2 = make_float2(0.5f * (sum_s[2 * cp] + sum_s[32 + 2 * cp]),
                                               0.5f * (sum_s[2 * cp + 1] + sum_s[32 + 2 * cp + 1]));  // 1/2 s
                const float2 c2 = make_float2(hs2.x + __uint_as_float((uint32_t)braw[0] << 16),
                                              hs2.y + __uint_as_float((uint32_t)braw[1] << 16));
                uint32_t* out_plane = reinterpret_cast<uint32_t*>(prm.out + plane_offset(prm.lo, bh, prm.hdiv)) + lane;
                const int sc = lane >> 1, sw = (lane & 1) * 8;
                const float* rq_l = rq_s + tp * kRqStride;  // the norm of the lane's token
                const uint32_t k_base = smem_u32(K_s) + cp * 4, z_addr = smem_u32(smem + kOffZero) + cp * 4;
                for (int u = ww; u < n_units; u += kWorkers / 32) {
                    const int y = u / segs, c0 = (u - y * segs) * kSeg, nc = min(kSeg, Wc - c0);
                    uint32_t ra[KS], rstep[KS];  // address of token (y + dy - R, 0) (or the zero row) and bytes per token
#pragma unroll
                    for (int dy = 0; dy < KS; ++dy) {
                        const int yy = y + dy - R;
                        const bool rv = (unsigned)yy < (unsigned)prm.gridH;
                        ra[dy] = rv ? k_base + (uint32_t)((prm.prefix + yy * W) * 64) : z_addr;
                        rstep[dy] = rv ? 64u : 0u;
                    }
#pragma unroll
                    for (int j = 0; j < kSeg; ++j) {
                        const int x = 2 * (c0 + j) + tp;  // the lane's token in the grid row
                        float2 part[KS];
#pragma unroll
                        for (int dy = 0; dy < KS; ++dy) {
                            part[dy] = (dy == 0) ? c2 : zero2;
#pragma unroll
                            for (int dx = 0; dx < KS; ++dx) {
                                const int xt = x + dx - R;
                                const uint32_t a = ((unsigned)xt < (unsigned)W) ? ra[dy] + (uint32_t)xt * rstep[dy] : z_addr;
                                uint32_t wv;
                                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(wv) : "r"(a));
                                part[dy] = ffma2(wreg[dy][dx], make_float2(bf16lo(wv), bf16hi(wv)), part[dy]);
                            }
                        }
                        float2 acc = part[0];
#pragma unroll
                        for (int dy = 1; dy < KS; ++dy) { acc.x += part[dy].x; acc.y += part[dy].y; }
                        const int pr = (prm.prefix + y * W) / 2 + c0 + j, tr = pr & (kTile - 1);  // row of the token pair
                        const uint8_t* srow = (pr < kTile ? V_s : Q_s) + tr * 256;
                        const float2 a2 = *reinterpret_cast<const float2*>(srow + ((sc ^ (tr & 7)) << 4) + sw);
                        const float rq = rq_l[pr];
                        const float2 o = ffma2(a2, make_float2(rq, rq), acc);
                        if (j < nc) out_plane[pr * (kD / 2)] = pack_bf16x2(o.x, o.y);
                    }
                }
                for (int pr = ww; pr < prm.prefix / 2; pr += kWorkers / 32) {  // off-grid leading tokens
                    const float2 a2 = *reinterpret_cast<const float2*>(V_s + pr * 256 + ((sc ^ (pr & 7)) << 4) + sw);
                    const float rq = rq_l[pr];
                    const float2 o = ffma2(a2, make_float2(rq, rq), hs2);
                    out_plane[pr * (kD / 2)] = pack_bf16x2(o.x, o.y);
                }
            } else {
                const float2 hs2 = make_float2(0.5f * sum_s[2 * lane], 0.5f * sum_s[2 * lane + 1]);  // 1/2 s
                const float2 c2 = make_float2(hs2.x + __uint_as_float((uint32_t)braw[0] << 16),
                                              hs2.y + __uint_as_float((uint32_t)braw[1] << 16));  // + bias: grid tokens
                uint32_t* out_plane = reinterpret_cast<uint32_t*>(prm.out + plane_offset(prm.lo, bh, prm.hdiv)) + lane;
                const long long out_tok = OUT_PACKED ? kD / 2 : prm.lo.token / 2;  // 32-bit words per token step
                const int sc = lane >> 1, sw = (lane & 1) * 8;  // chunk and offset of the lane's pair in an fp32 row
                const float* rq_l = rq_s + ((prm.blockdiag && lane >= 16) ? kRqStride : 0);  // the norm of the lane's head
                // Branch-free inside a unit: a neighbour outside the grid is read from a row of zeros, the
                // columns of a ragged last unit are computed (from in-bounds shared memory) and not stored.
                const uint32_t k_base = smem_u32(K_s) + lane * 4, z_addr = smem_u32(smem + kOffZero) + lane * 4;
                for (int u = ww; u < n_units; u += kWorkers / 32) {
                    const int y = u / segs, x0 = (u - y * segs) * kSeg, nx = min(kSeg, W - x0);
                    uint32_t ra[KS];  // address of the lane's word of token (y + dy - R, x0); rows outside the grid: the zero row
                    uint32_t rstep[KS];  // bytes per column in that row (0 for the zero row)
    #pragma unroll
                    for (int dy = 0; dy < KS; ++dy) {
                        const int yy = y + dy - R;
                        const bool rv = (unsigned)yy < (unsigned)prm.gridH;
                        ra[dy] = rv ? k_base + (uint32_t)((prm.prefix + yy * W + x0) * 128) : z_addr;
                        rstep[dy] = rv ? 128u : 0u;
                    }
                    float2 win[KS][KS];  // column x0 - R + jj lives in slot jj % KS
    #pragma unroll
                    for (int jj = 0; jj < KS - 1 + kSeg; ++jj) {
                        // load column jj of the window (grid column x0 - R + jj), then finish output column jj - (KS - 1)
                        const bool cv = (unsigned)(x0 + jj - R) < (unsigned)W;
    #pragma unroll
                        for (int dy = 0; dy < KS; ++dy) {
                            const uint32_t a = cv ? ra[dy] + (uint32_t)(jj - R) * rstep[dy] : z_addr;
                            uint32_t wv;
                            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(wv) : "r"(a));
                            win[dy][jj % KS] = make_float2(bf16lo(wv), bf16hi(wv));
                        }
                        if (jj >= KS - 1) {  // compile-time
                            const int j = jj - (KS - 1);
                            float2 part[KS];  // one chain per filter row
    #pragma unroll
                            for (int dy = 0; dy < KS; ++dy) {
                                part[dy] = (dy == 0) ? c2 : zero2;
    #pragma unroll
                                for (int dx = 0; dx < KS; ++dx) part[dy] = ffma2(wreg[dy][dx], win[dy][(j + dx) % KS], part[dy]);
                            }
                            float2 acc = part[0];
    #pragma unroll
                            for (int dy = 1; dy < KS; ++dy) { acc.x += part[dy].x; acc.y += part[dy].y; }
                            const int t = prm.prefix + y * W + x0 + j, tr = t & (kTile - 1);  // t < N + kSeg: inside a row of rq_s
                            const uint8_t* srow = (t < kTile ? V_s : Q_s) + tr * 256;
                            const float2 a2 = *reinterpret_cast<const float2*>(srow + ((sc ^ (tr & 7)) << 4) + sw);
                            const float rq = rq_l[t];
                            const float2 o = ffma2(a2, make_float2(rq, rq), acc);
                            if (j < nx) out_plane[t * out_tok] = pack_bf16x2(o.x, o.y);
                        }
                    }
                }
                // off-grid leading tokens: the attention terms only
                for (int t = ww; t < prm.prefix; t += kWorkers / 32) {
                    const float2 a2 = *reinterpret_cast<const float2*>(V_s + t * 256 + ((sc ^ (t & 7)) << 4) + sw);
                    const float rq = rq_l[t];
                    const float2 o = ffma2(a2, make_float2(rq, rq), hs2);
                    out_plane[t * out_tok] = pack_bf16x2(o.x, o.y);
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(plane_free);
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

template <int KS>
cudaError_t launch_fused_ks(const Problem& p, unsigned* status, cudaStream_t st) {
    CUtensorMap tmK, tmV, tmQ, tmVplain;
    // [64, tokens, planes per batch step, batch steps]
    const uint64_t nb = (uint64_t)(p.BH / p.hdiv);
    const bool pair = (p.d == 32);  // two tokens per 128-byte row
    const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)(pair ? p.N / 2 : p.N), (uint64_t)p.hdiv, nb};
    const uint32_t box[4] = {kD, kTile, 1, 1};
    auto strides = [&](const Layout& l, uint64_t (&s)[3]) {
        s[0] = (uint64_t)(pair ? kD : l.token); s[1] = (uint64_t)l.head; s[2] = (uint64_t)(nb > 1 ? l.batch : l.head * p.hdiv);
    };
    uint64_t sq[3], sk[3], sv[3];
    strides(p.lq, sq); strides(p.lk, sk); strides(p.lv, sv);
    if (!make_tensor_map_bf16(&tmK, p.k, 4, dims, sk, box, true) || !make_tensor_map_bf16(&tmV, p.v, 4, dims, sv, box, true) ||
        !make_tensor_map_bf16(&tmQ, p.q, 4, dims, sq, box, true) || !make_tensor_map_bf16(&tmVplain, p.v, 4, dims, sv, box, false))
        return cudaErrorNotSupported;
    FusedParams prm;
    prm.w = static_cast<const __nv_bfloat16*>(p.w);
    prm.bias = static_cast<const __nv_bfloat16*>(p.bias);
    prm.out = static_cast<__nv_bfloat16*>(p.out);
    prm.lo = p.lo;
    prm.blockdiag = p.blockdiag ? 1 : 0;
    prm.H = p.H; prm.head0 = p.head0; prm.BH = p.BH; prm.hdiv = p.hdiv; prm.prefix = p.prefix; prm.N = p.N;
    prm.gridH = p.gridH; prm.gridW = p.gridW;
    prm.eps2 = p.eps2; prm.status = status;
    static PerDevice opt_in[3];  // per instantiation
    const bool packed = (p.lo.token == kD);
    const cudaError_t e = pair     ? opt_in_smem(tc_fused_kernel<KS, true, true>, kSmemBytes, opt_in[2])
                          : packed ? opt_in_smem(tc_fused_kernel<KS, true, false>, kSmemBytes, opt_in[1])
                                   : opt_in_smem(tc_fused_kernel<KS, false, false>, kSmemBytes, opt_in[0]);
    if (e != cudaSuccess) return e;
    const int resident = 2 * device_sm_count();  // two CTAs per multiprocessor
    const int grid = p.BH < resident ? p.BH : resident;
    if (pair)
        tc_fused_kernel<KS, true, true><<<(unsigned)grid, kThreads, kSmemBytes, st>>>(tmK, tmV, tmQ, tmVplain, prm);
    else if (packed)
        tc_fused_kernel<KS, true, false><<<(unsigned)grid, kThreads, kSmemBytes, st>>>(tmK, tmV, tmQ, tmVplain, prm);
    else
        tc_fused_kernel<KS, false, false><<<(unsigned)grid, kThreads, kSmemBytes, st>>>(tmK, tmV, tmQ, tmVplain, prm);
    return cudaGetLastError();
}

}  // namespace

bool fused_supports(const Problem& p) {
    if (!p.bf16 || (p.ksize != 3 && p.ksize != 5)) return false;
    if (p.d == kD) return p.N <= kMaxTiles * kTile;
    return token_pairs(p) && p.prefix % 2 == 0 && p.N / 2 <= kMaxTiles * kTile;  // width 32: rows of two tokens
}

cudaError_t launch_fused(const Problem& p, unsigned* status, cudaStream_t st) {
    return p.ksize == 3 ? launch_fused_ks<3>(p, status, st) : launch_fused_ks<5>(p, status, st);
}

}  // namespace tc
}  // namespace castling

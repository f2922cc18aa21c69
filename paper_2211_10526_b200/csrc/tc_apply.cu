// Apply kernel of the tensor-core path (bf16; width-64 heads, or width-32 heads packed two to a 128-byte
// row: see the modes at the kernel template):
//     out_t = (1/pi) q^_t S + 1/2 s + bias + DWConv(V)_t                         (Eq. 9)
// Persistent CTAs walk a contiguous range of 8 x 16-token patches of the token grid.  Per patch
//   warp 0      TMA: the raw Q patch (128 rows of 128 B, 128-byte swizzle) and the V patch with
//               its halo; out-of-grid rows and columns are zero-filled by TMA, which is exactly
//               the convolution's zero padding
//   warp 1      one thread issues four UMMAs: acc[128 x 64] = Q[128 x 64] * S'[64 x 64] into TMEM,
//               S' = S / pi in bf16; the row scale 1/||q|| commutes and is applied afterwards
//   warps 10..17 depthwise convolution on CUDA cores, one lane per channel pair, filters in
//               registers, sliding window along x (two rows x eight columns per warp), packed
//               fp32x2 FMAs, result (+ 1/2 s + bias) staged in shared memory as fp32
//   warps 2..9  one thread per token and half of its channels: ||q|| from the Q patch (each of
//               the two warps of a token sums half of the row, exchanged through shared memory),
//               accumulator row from TMEM, out = acc / max(||q||, eps) + staged, one rounding to
//               bf16, patch written to shared memory and stored with TMA (clipped at the grid edge)
#include "tc_common.cuh"
#include "tc_host.cuh"

namespace castling {
namespace tc {
namespace {

constexpr int kD = 64;
constexpr int kTY = 8, kTX = 16;            // patch: 8 rows x 16 columns = 128 tokens
constexpr int kTile = kTY * kTX;
constexpr int kQBytes = kTile * kD * 2;     // 16 KiB
constexpr int kStgStride = kD * 4 + 16;     // fp32 row + 16 B pad: conflict-free row-per-thread reads
constexpr int kStgBytes = kTile * kStgStride;
constexpr int kEpiWarps = 8;                   // two warps per TMEM lane quarter
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kTmemCols = 128;              // two 64-column accumulators

// PAIR = true serves head width 32: a 128-byte row holds two horizontally adjacent tokens, so a
// "column" of the patch is a token pair and the 8 x 16-column patch covers 8 x 32 tokens.
template <int KS, bool PAIR> struct Geo {
    // conv warps: each takes kConvRows patch rows x 8 columns.  3x3: 8 warps of 2 rows; 5x5: 4 warps of
    // 4 rows (fewer redundant window loads, and the larger window fits the registers of 448 threads)
    static constexpr int kConvRows = (KS == 3) ? 2 : 4;
    static constexpr int kConvWarps = 2 * kTY / kConvRows, kConvThreads = kConvWarps * 32;
    static constexpr int kThreads = 64 + kEpiThreads + kConvThreads;
    static constexpr int R = KS / 2;
    static constexpr int HC = PAIR ? (R + 1) / 2 : R;   // halo columns on each side
    static constexpr int HY = kTY + 2 * R, HX = kTX + 2 * HC;
    static constexpr int kVBytes = HY * HX * kD * 2;
    static constexpr int kStage = ((kQBytes + kVBytes + 1023) / 1024) * 1024;
    static constexpr int kStages = (KS == 3) ? 3 : 2;
    // S' | out patch | stages | staging x2 | rq x2 | barriers
    static constexpr int kOffS = 0, kOffOut = 8192, kOffStages = kOffOut + kQBytes;
    static constexpr int kOffStg = kOffStages + kStages * kStage;
    static constexpr int kOffRq = kOffStg + 2 * kStgBytes;   // sum of squares of each half of a Q row
    static constexpr int kOffBar = kOffRq + 2 * kTile * 4;
    static constexpr size_t kSmem = 1024 + kOffBar + 256;
    // row-sum normalisation: a second 64-wide block of the operand (its first columns hold sum k^ / pi) and 1/2 s per
    // staging buffer
    static constexpr int kOffS2 = ((kOffBar + 256 + 1023) / 1024) * 1024, kOffHs = kOffS2 + 8192;
    static constexpr size_t kSmemRN = 1024 + kOffHs + 2 * kD * 4;
};

struct ApplyParams {
    const float* state;            // [BH][P][64*64 + 64] raw sums of the P token splits
    int P;
    const __nv_bfloat16* w;        // [H*d][KS][KS]
    const __nv_bfloat16* bias;     // [H*d] or nullptr
    int flat;                      // the planes have one uniform stride: the tensor maps are 4-D, [.., plane]
    int H, head0, bh0, hdiv, tilesX, tilesY, n_tiles;  // tiles of (b,h) in [bh0, bh0 + n_tiles / (tilesX*tilesY))
    float eps2;
    unsigned* status;
    int v_row0;                    // V holds more grid rows than the plane has (a band of a sharded sequence with its
                                   // neighbours' rows): its row v_row0 is grid row 0
    int n_tokens;                  // tokens per sequence (row-sum normalisation: the sum of the constant 1/2 terms is n_tokens / 2)
};

// Position of a CTA's current patch, advanced without divisions (one step per patch in every role).
struct PatchWalk {
    int bh, py, px;
    __device__ __forceinline__ PatchWalk(int g, int tilesX, int tilesY) {
        const int per = tilesX * tilesY;
        bh = g / per;
        const int rem = g - bh * per;
        py = rem / tilesX;
        px = rem - py * tilesX;
    }
    __device__ __forceinline__ void step(int tilesX, int tilesY) {
        if (++px == tilesX) { px = 0; if (++py == tilesY) { py = 0; ++bh; } }
    }
};

// MODE 0: width-64 heads; 1: width-32 heads, two adjacent tokens per 128-byte row (the PAIR geometry);
// 2: two width-32 heads side by side in the one-token-per-row geometry (block-diagonal state).
// RN: row-sum normalisation (Eq. 3's denominator on the kept kernel of Eq. 8).  The state carries sum_n k^_n behind s; the
// operand gets one or two more columns (sum k^ / pi per head or token of the row), so that column 64 (65) of the
// accumulator is q . sum k^ / pi; the attention term (acc / ||q|| + 1/2 s) is divided by n_tokens / 2 + that product
// / ||q|| before the convolution and the bias are added.
template <int KS, int MODE, bool RN>
__global__ void __launch_bounds__((Geo<KS, MODE == 1>::kThreads), 1)
tc_apply_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmO, const ApplyParams prm) {
    constexpr bool PAIR = (MODE == 1), BLOCKDIAG = (MODE == 2);
    using G = Geo<KS, PAIR>;
    constexpr int NS = G::kStages;
    constexpr int kSW = kD * kD + kD + (RN ? kD : 0);   // words of one state
    constexpr int kAcc = RN ? 2 * kD : kD;              // TMEM columns per accumulator
    constexpr int kAccN = RN ? kD + 16 : kD;            // columns the UMMAs write
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* S_s = smem + G::kOffS;
    uint8_t* out_s = smem + G::kOffOut;
    uint8_t* stages = smem + G::kOffStages;
    uint8_t* stg = smem + G::kOffStg;
    float* rq_s = reinterpret_cast<float*>(smem + G::kOffRq);
    uint8_t* S2_s = smem + G::kOffS2;                                  // RN only
    float* hs_s = reinterpret_cast<float*>(smem + G::kOffHs);          // RN only: [2][64]
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + G::kOffBar);  // [NS] TMA landed
    uint64_t* empty = full + NS;                                      // [NS] stage consumed (conv + epilogue warps, UMMA commit)
    uint64_t* acc_full = empty + NS;                                  // [2]  UMMAs retired
    uint64_t* conv_full = acc_full + 2;                               // [2]  staging written (conv warps)
    uint64_t* buf_free = conv_full + 2;                               // [2]  accumulator + staging read (128)
    uint64_t* s_ready = buf_free + 2;                                 // S' of the current (b,h) written (128)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_ready + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // contiguous share of the patches for this CTA
    const int g_begin = (int)((long long)prm.n_tiles * blockIdx.x / gridDim.x);
    const int g_end = (int)((long long)prm.n_tiles * (blockIdx.x + 1) / gridDim.x);
    const int my_tiles = g_end - g_begin;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], G::kConvThreads + kEpiThreads + 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&conv_full[b], G::kConvThreads); mbar_init(&buf_free[b], kEpiThreads); }
        mbar_init(s_ready, kEpiThreads);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmO);
    }
    if (warp == 1) tmem_alloc(tmem_slot, RN ? 2 * kTmemCols : kTmemCols);
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    constexpr unsigned kBit = kStatusApplyTimeout;
    // the next forward's state kernel (launched programmatically dependent) may set itself up on multiprocessors
    // this grid has left; it waits for this grid's completion before it touches global memory
    pdl_launch_dependents();

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            const uint64_t pol_q = l2_policy_evict_first();  // Q is read once
            PatchWalk pw(g_begin, prm.tilesX, prm.tilesY);
            for (int it = 0; it < my_tiles; ++it, pw.step(prm.tilesX, prm.tilesY)) {
                const int s = it % NS, use = it / NS;
                if (use > 0 && !mbar_wait(&empty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) break;
                const int bh = pw.bh, y0 = pw.py * kTY, x0 = pw.px * kTX;
                uint8_t* qs = stages + s * G::kStage;
                mbar_expect_tx(&full[s], kQBytes + G::kVBytes);
                if (prm.flat) {
                    tma_load_4d_hint(qs, &tmQ, &full[s], 0, x0, y0, bh, pol_q);
                    tma_load_4d(qs + kQBytes, &tmV, &full[s], 0, x0 - G::HC, y0 - G::R + prm.v_row0, bh);
                } else {
                    const int pb = bh / prm.hdiv, ph = bh - pb * prm.hdiv;
                    tma_load_5d_hint(qs, &tmQ, &full[s], 0, x0, y0, ph, pb, pol_q);
                    tma_load_5d(qs + kQBytes, &tmV, &full[s], 0, x0 - G::HC, y0 - G::R + prm.v_row0, ph, pb);
                }
                ++issued;
            }
            if (*abort_flag) {
                for (int i = max(0, issued - NS); i < issued; ++i)
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&full[i % NS], (i / NS) & 1); ++spin) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, kAccN, false, true);
            const uint32_t s_addr = smem_u32(S_s);
            const uint32_t lbo = RN ? smem_u32(S2_s) - s_addr : 0;     // to the operand's second 64-wide block
            int prev_bh = -1, seg = 0;
            PatchWalk pw(g_begin, prm.tilesX, prm.tilesY);
            for (int it = 0; it < my_tiles; ++it, pw.step(prm.tilesX, prm.tilesY)) {
                const int s = it % NS, use = it / NS, b = it & 1, ub = it >> 1;
                const int bh = pw.bh;
                if (bh != prev_bh) {
                    if (!mbar_wait(s_ready, seg & 1, abort_flag, prm.status, kBit)) break;
                    ++seg; prev_bh = bh;
                }
                if (!mbar_wait(&full[s], use & 1, abort_flag, prm.status, kBit)) break;
                if (ub > 0 && !mbar_wait(&buf_free[b], (ub - 1) & 1, abort_flag, prm.status, kBit)) break;
                tcgen05_fence_after_sync();
                const uint32_t q_addr = smem_u32(stages + s * G::kStage);
#pragma unroll
                for (int k = 0; k < kD / 16; ++k) {
                    const uint64_t a = umma_desc_sw128(q_addr + k * 32, 0, 1024);        // K-major rows of 128 B
                    const uint64_t bd = umma_desc_sw128(s_addr + k * 2048, lbo, 1024);   // N-major, 16 K-rows per step
                    umma_bf16(tmem + b * kAcc, a, bd, idesc, k != 0);
                }
                umma_commit(&acc_full[b]);
                umma_commit(&empty[s]);  // the same UMMAs have finished reading the Q patch
            }
        }
    } else if (warp < 2 + kEpiWarps) {
        // ------- epilogue: thread = (token of the patch, half of the channels) -------
        const int quarter = warp & 3, row = quarter * 32 + lane, et = tid - 64;
        const int half = (warp - 2) >> 2;  // channels half*32 .. half*32 + 31
        const bool leader = (et == 0);
        const uint64_t pol_o = l2_policy_evict_first();  // the output is not read back here
        int prev_bh = -1;
        pdl_wait_primary();  // the state kernel's results are read below
        PatchWalk pw(g_begin, prm.tilesX, prm.tilesY);
        for (int it = 0; it < my_tiles; ++it, pw.step(prm.tilesX, prm.tilesY)) {
            const int b = it & 1, ub = it >> 1;
            const int bh = pw.bh, y0 = pw.py * kTY, x0 = pw.px * kTX;
            if (bh != prev_bh) {
                // every UMMA that read the previous S' has retired (its acc_full was waited on below)
                prev_bh = bh;
                const int i = et >> 2, part = et & 3;  // row i of the operand, 16 columns part*16 ..
                const float* st = prm.state + (size_t)(prm.bh0 + bh) * prm.P * kSW;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    float4 lo, hi;
                    if (!PAIR) {
                        const float4* src = reinterpret_cast<const float4*>(st + i * kD + part * 16);
                        lo = __ldg(src + 2 * c); hi = __ldg(src + 2 * c + 1);
                        for (int pp = 1; pp < prm.P; ++pp) {  // fixed order: bitwise reproducible
                            const float4 l2 = __ldg(src + pp * (kSW / 4) + 2 * c);
                            const float4 h2 = __ldg(src + pp * (kSW / 4) + 2 * c + 1);
                            lo.x += l2.x; lo.y += l2.y; lo.z += l2.z; lo.w += l2.w;
                            hi.x += h2.x; hi.y += h2.y; hi.z += h2.z; hi.w += h2.w;
                        }
                        if (BLOCKDIAG && ((i < 32) != (part < 2))) {  // off-diagonal block: the other head's keys
                            lo = make_float4(0.f, 0.f, 0.f, 0.f); hi = lo;
                        }
                    } else {
                        // operand = blockdiag(S32, S32) with S32 = block(0,0) + block(1,1) of the paired sums
                        const int col = part * 16 + c * 8;  // first of 8 columns
                        if ((i < 32) == (col < 32)) {
                            const int a = i & 31, bcol = col & 31;
                            const float4* s0 = reinterpret_cast<const float4*>(st + a * kD + bcol);
                            const float4* s1 = reinterpret_cast<const float4*>(st + (32 + a) * kD + 32 + bcol);
                            const float4 l0 = __ldg(s0), h0 = __ldg(s0 + 1), l1 = __ldg(s1), h1 = __ldg(s1 + 1);
                            lo = make_float4(l0.x + l1.x, l0.y + l1.y, l0.z + l1.z, l0.w + l1.w);
                            hi = make_float4(h0.x + h1.x, h0.y + h1.y, h0.z + h1.z, h0.w + h1.w);
                        } else {
                            lo = make_float4(0.f, 0.f, 0.f, 0.f); hi = lo;
                        }
                    }
                    uint4 o;
                    o.x = pack_bf16x2(lo.x * kInvPi, lo.y * kInvPi); o.y = pack_bf16x2(lo.z * kInvPi, lo.w * kInvPi);
                    o.z = pack_bf16x2(hi.x * kInvPi, hi.y * kInvPi); o.w = pack_bf16x2(hi.z * kInvPi, hi.w * kInvPi);
                    *reinterpret_cast<uint4*>(S_s + i * 128 + (((part * 2 + c) ^ (i & 7)) << 4)) = o;
                    if (RN) {
                        // second block of the operand: row i (a key feature) holds sum k^[i] / pi in column 0, or, where a
                        // row carries two tokens or two heads, in the column of its half; the rest is zero
                        uint4 z = make_uint4(0, 0, 0, 0);
                        if (part == 0 && c == 0) {
                            const float* sk = st + kD * kD + kD;
                            float val;
                            if (PAIR) val = __ldg(sk + (i & 31)) + __ldg(sk + 32 + (i & 31));   // both token parities
                            else val = __ldg(sk + i);
                            const uint32_t hv = pack_bf16x2(val * kInvPi, 0.f) & 0xffffu;
                            z.x = (MODE != 0 && i >= 32) ? (hv << 16) : hv;
                        }
                        *reinterpret_cast<uint4*>(S2_s + i * 128 + (((part * 2 + c) ^ (i & 7)) << 4)) = z;
                    }
                }
                fence_proxy_async_smem();
                mbar_arrive(s_ready);
            }
            {   // this thread's half of sum(q^2) for its token; the other half comes from the partner warp
                const int s = it % NS, use = it / NS;
                if (!mbar_wait(&full[s], use & 1, abort_flag, prm.status, kBit)) break;
                const uint8_t* qrow = stages + s * G::kStage + row * 128;
                float ss[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 c = *reinterpret_cast<const uint4*>(qrow + (((4 * half + j) ^ (row & 7)) << 4));
                    const uint32_t w4[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float lo = bf16lo(w4[e]), hi = bf16hi(w4[e]);
                        ss[e] = fmaf(lo, lo, ss[e]); ss[e] = fmaf(hi, hi, ss[e]);
                    }
                }
                rq_s[half * kTile + row] = (ss[0] + ss[1]) + (ss[2] + ss[3]);
                mbar_arrive(&empty[s]);  // the Q rows of this stage have been read
            }
            if (!mbar_wait(&acc_full[b], ub & 1, abort_flag, prm.status, kBit)) break;
            tcgen05_fence_after_sync();
            float a[32];
            {
                float a0[16], a1[16];
                tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + b * kAcc + half * 32, a0);
                tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + b * kAcc + half * 32 + 16, a1);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 16; ++e) { a[e] = a0[e]; a[16 + e] = a1[e]; }
            }
            float qk = 0.f;  // RN: q . sum k^ / pi of this thread's token
            if (RN) {
                float x[16];
                tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + b * kAcc + kD, x);
                tmem_ld_wait();
                qk = (MODE != 0 && half == 1) ? x[1] : x[0];
            }
            if (!mbar_wait(&conv_full[b], ub & 1, abort_flag, prm.status, kBit)) break;
            // the previous patch's TMA store must have read out_s before it is rewritten; the same
            // barrier makes both halves of every row's sum of squares visible
            if (it > 0 && leader) tma_store_wait_read();
            named_barrier_sync(1, kEpiThreads);
            const float rq = (PAIR || BLOCKDIAG)
                                 ? rsqrtf(fmaxf(rq_s[half * kTile + row], prm.eps2))   // half row = one token / one head
                                 : rsqrtf(fmaxf(rq_s[row] + rq_s[kTile + row], prm.eps2));
            const uint8_t* srow = stg + b * kStgBytes + row * kStgStride + half * 128;
            uint8_t* orow = out_s + row * 128;
            if (RN) {
                // (acc / ||q|| + 1/2 s) / (n / 2 + q^ . sum k^ / pi); the staged value is convolution + bias only
                const float inv = 1.0f / fmaf(qk, rq, 0.5f * (float)prm.n_tokens);
                const float* hrow = hs_s + b * kD + half * 32;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float4 hv = *reinterpret_cast<const float4*>(hrow + 4 * e);
                    a[4 * e + 0] = fmaf(a[4 * e + 0], rq, hv.x) * inv; a[4 * e + 1] = fmaf(a[4 * e + 1], rq, hv.y) * inv;
                    a[4 * e + 2] = fmaf(a[4 * e + 2], rq, hv.z) * inv; a[4 * e + 3] = fmaf(a[4 * e + 3], rq, hv.w) * inv;
                }
            }
            const float rqm = RN ? 1.0f : rq;  // RN: the scale has been applied above
#pragma unroll
            for (int e = 0; e < 4; ++e) {  // 8 channels -> one 16-byte chunk of the bf16 row
                const float4 c0 = *reinterpret_cast<const float4*>(srow + e * 32);
                const float4 c1 = *reinterpret_cast<const float4*>(srow + e * 32 + 16);
                uint4 pk;
                pk.x = pack_bf16x2(fmaf(a[8 * e + 0], rqm, c0.x), fmaf(a[8 * e + 1], rqm, c0.y));
                pk.y = pack_bf16x2(fmaf(a[8 * e + 2], rqm, c0.z), fmaf(a[8 * e + 3], rqm, c0.w));
                pk.z = pack_bf16x2(fmaf(a[8 * e + 4], rqm, c1.x), fmaf(a[8 * e + 5], rqm, c1.y));
                pk.w = pack_bf16x2(fmaf(a[8 * e + 6], rqm, c1.z), fmaf(a[8 * e + 7], rqm, c1.w));
                *reinterpret_cast<uint4*>(orow + (((half * 4 + e) ^ (row & 7)) << 4)) = pk;
            }
            tcgen05_fence_before_sync();
            mbar_arrive(&buf_free[b]);
            fence_proxy_async_smem();
            named_barrier_sync(1, kEpiThreads);
            if (leader) {
                if (prm.flat) {
                    tma_store_4d_hint(&tmO, out_s, 0, x0, y0, bh, pol_o);
                } else {
                    const int pb = bh / prm.hdiv;
                    tma_store_5d_hint(&tmO, out_s, 0, x0, y0, bh - pb * prm.hdiv, pb, pol_o);
                }
                tma_store_commit();
            }
        }
        if (leader) tma_store_wait_all();
    } else {
        // ------- depthwise convolution: lane = channel pair, warp = two patch rows x eight columns -------
        const int cw = (warp - 2 - kEpiWarps) >> 1, xh = (warp - 2 - kEpiWarps) & 1;
        constexpr int kCX = kTX / 2;
        constexpr int R = G::R, RO = G::kConvRows, ROWS = RO + 2 * R;
        float2 wreg[KS][KS];
        float2 cinit = make_float2(0.f, 0.f), hs2 = make_float2(0.f, 0.f);
        int prev_bh = -1;
        pdl_wait_primary();  // the token sums of the state kernel are read below
        PatchWalk pw(g_begin, prm.tilesX, prm.tilesY);
        for (int it = 0; it < my_tiles; ++it, pw.step(prm.tilesX, prm.tilesY)) {
            const int s = it % NS, use = it / NS, b = it & 1, ub = it >> 1;
            const int bh = pw.bh;
            if (bh != prev_bh) {
                prev_bh = bh;
                // this lane's channel pair: 2*lane of 64 channels, or (PAIR) 2*(lane & 15) of 32 channels
                // for the token of parity lane >> 4
                const int gbh = prm.bh0 + bh;
                const int cp2 = PAIR ? 2 * (lane & 15) : 2 * lane;
                const int ch = ((prm.head0 + gbh) % prm.H) * (PAIR ? 32 : kD) + cp2;
                const float* sv = prm.state + (size_t)gbh * prm.P * kSW + kD * kD;
                float s0, s1;
                if (PAIR) {  // token sum = sum of the two halves of the paired sums
                    s0 = __ldg(sv + cp2) + __ldg(sv + 32 + cp2);
                    s1 = __ldg(sv + cp2 + 1) + __ldg(sv + 32 + cp2 + 1);
                } else {
                    s0 = __ldg(sv + cp2); s1 = __ldg(sv + cp2 + 1);
                    for (int pp = 1; pp < prm.P; ++pp) {
                        s0 += __ldg(sv + pp * kSW + cp2);
                        s1 += __ldg(sv + pp * kSW + cp2 + 1);
                    }
                }
                cinit.x = RN ? 0.f : 0.5f * s0; cinit.y = RN ? 0.f : 0.5f * s1;
                hs2 = make_float2(0.5f * s0, 0.5f * s1);
                if (prm.bias) { cinit.x += __bfloat162float(prm.bias[ch]); cinit.y += __bfloat162float(prm.bias[ch + 1]); }
#pragma unroll
                for (int dy = 0; dy < KS; ++dy)
#pragma unroll
                    for (int dx = 0; dx < KS; ++dx)
                        wreg[dy][dx] = make_float2(__bfloat162float(prm.w[(size_t)ch * KS * KS + dy * KS + dx]),
                                                   __bfloat162float(prm.w[(size_t)(ch + 1) * KS * KS + dy * KS + dx]));
            }
            if (!mbar_wait(&full[s], use & 1, abort_flag, prm.status, kBit)) break;
            if (ub > 0 && !mbar_wait(&buf_free[b], (ub - 1) & 1, abort_flag, prm.status, kBit)) break;
            // Window of KS tokens per halo row, sliding along x.  Token t (relative to the first token this
            // lane needs) sits U bytes after token t-1: U = 128, one token per column, or (PAIR) 64.
            // One output column advances the window by STEP tokens (2 when PAIR: the lane's token keeps
            // its parity).  Slot of token t in the rotating window: t % KS (t is a compile-time value).
            constexpr int U = PAIR ? 64 : 128, STEP = PAIR ? 2 : 1;
            const int tok0 = PAIR ? 2 * (xh * kCX + G::HC) + (lane >> 4) - R : xh * kCX;
            const uint8_t* vh = stages + s * G::kStage + kQBytes + (RO * cw) * G::HX * 128 + tok0 * U +
                                (PAIR ? (lane & 15) * 4 : lane * 4);
            uint8_t* so = stg + b * kStgBytes + ((RO * cw) * kTX + xh * kCX) * kStgStride + lane * 8;
            float2 win[ROWS][KS];
#pragma unroll
            for (int t = 0; t < KS - STEP; ++t)
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    const uint32_t wv = *reinterpret_cast<const uint32_t*>(vh + r * G::HX * 128 + t * U);
                    win[r][t % KS] = make_float2(bf16lo(wv), bf16hi(wv));
                }
#pragma unroll
            for (int x = 0; x < kCX; ++x) {
#pragma unroll
                for (int n = 0; n < STEP; ++n) {
                    const int t = STEP * x + KS - STEP + n;  // compile-time after unrolling
#pragma unroll
                    for (int r = 0; r < ROWS; ++r) {
                        const uint32_t wv = *reinterpret_cast<const uint32_t*>(vh + r * G::HX * 128 + t * U);
                        win[r][t % KS] = make_float2(bf16lo(wv), bf16hi(wv));
                    }
                }
                float2 acc[RO];
#pragma unroll
                for (int r = 0; r < RO; ++r) acc[r] = cinit;
#pragma unroll
                for (int dy = 0; dy < KS; ++dy)
#pragma unroll
                    for (int dx = 0; dx < KS; ++dx)
#pragma unroll
                        for (int r = 0; r < RO; ++r)
                            acc[r] = ffma2(wreg[dy][dx], win[dy + r][(STEP * x + dx) % KS], acc[r]);
#pragma unroll
                for (int r = 0; r < RO; ++r) *reinterpret_cast<float2*>(so + (r * kTX + x) * kStgStride) = acc[r];
            }
            if (RN && cw == 0 && xh == 0) {
                // 1/2 s of the plane this patch belongs to, per column of a 128-byte row, beside the staging buffer
                const int col = PAIR ? (lane >> 4) * 32 + 2 * (lane & 15) : 2 * lane;
                *reinterpret_cast<float2*>(hs_s + b * kD + col) = hs2;
            }
            mbar_arrive(&empty[s]);      // the V patch of this stage is no longer needed
            mbar_arrive(&conv_full[b]);
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, RN ? 2 * kTmemCols : kTmemCols);
}

template <int KS, int MODE, bool RN>
cudaError_t launch_apply_ks(const Problem& p, const float* state, int P, unsigned* status, cudaStream_t st) {
    constexpr bool PAIR = (MODE == 1);
    using G = Geo<KS, PAIR>;
    CUtensorMap tmQ, tmV, tmO;
    const int cols = PAIR ? p.gridW / 2 : p.gridW;  // 128-byte columns per grid row
    // [64, columns, grid rows, planes per batch step, batch steps]; with a single batch step the last
    // dimension is dropped (a 4-D copy is a little cheaper for the TMA unit than a 5-D one)
    const uint64_t nb = (uint64_t)(p.BH / p.hdiv);
    const int rank = nb > 1 ? 5 : 4;
    const uint64_t dims[5] = {(uint64_t)kD, (uint64_t)cols, (uint64_t)p.gridH, (uint64_t)p.hdiv, nb};
    const uint32_t box[5] = {kD, kTX, kTY, 1, 1};
    const uint32_t boxv[5] = {kD, (uint32_t)G::HX, (uint32_t)G::HY, 1, 1};
    auto strides = [&](const Layout& l, uint64_t (&s)[4]) {
        s[0] = (uint64_t)(PAIR ? kD : l.token);          // next column: one token, or (PAIR) two
        s[1] = (uint64_t)(l.token * p.gridW);            // next grid row
        s[2] = (uint64_t)l.head;
        s[3] = (uint64_t)(nb > 1 ? l.batch : l.head * p.hdiv);
    };
    uint64_t sq[4], sv[4], so[4];
    strides(p.lq, sq); strides(p.lv, sv); strides(p.lo, so);
    // the token grid starts after the off-grid leading tokens of every plane
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + p.prefix * p.lq.token;
    const __nv_bfloat16* vg = static_cast<const __nv_bfloat16*>(p.v) + p.prefix * p.lv.token;
    __nv_bfloat16* og = static_cast<__nv_bfloat16*>(p.out) + p.prefix * p.lo.token;
    // V may hold more grid rows than the plane (the neighbours' rows of a band of a sharded sequence): rows outside
    // that taller tensor, not outside the band, are the zero padding
    uint64_t dimsv[5] = {dims[0], dims[1], (uint64_t)(p.v_rows > 0 ? p.v_rows : p.gridH), dims[3], dims[4]};
    if (!make_tensor_map_bf16(&tmQ, qg, rank, dims, sq, box, true) || !make_tensor_map_bf16(&tmO, og, rank, dims, so, box, true) ||
        !make_tensor_map_bf16(&tmV, vg, rank, dimsv, sv, boxv, false))
        return cudaErrorNotSupported;
    ApplyParams prm;
    prm.state = state;
    prm.P = P;
    prm.w = static_cast<const __nv_bfloat16*>(p.w);
    prm.bias = static_cast<const __nv_bfloat16*>(p.bias);
    prm.flat = (rank == 4) ? 1 : 0;
    prm.H = p.H; prm.head0 = p.head0; prm.bh0 = 0; prm.hdiv = p.hdiv;
    prm.tilesX = (cols + kTX - 1) / kTX; prm.tilesY = (p.gridH + kTY - 1) / kTY;
    prm.n_tiles = p.BH * prm.tilesX * prm.tilesY;
    prm.eps2 = p.eps2; prm.status = status; prm.n_tokens = p.N; prm.v_row0 = p.v_rows > 0 ? p.v_row0 : 0;
    constexpr size_t kSmemBytes = RN ? G::kSmemRN : G::kSmem;
    static PerDevice opt_in;  // one per instantiation
    {
        const cudaError_t e = opt_in_smem(tc_apply_kernel<KS, MODE, RN>, kSmemBytes, opt_in);
        if (e != cudaSuccess) return e;
    }
    const int sms = device_sm_count();  // one persistent CTA per multiprocessor
    const int grid = prm.n_tiles < sms ? prm.n_tiles : sms;
    // programmatic dependent launch: this grid's prologue and first Q / V loads overlap the tail of
    // the state kernel; the warps that read its results wait for it (griddepcontrol.wait) first
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(G::kThreads); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc_apply_kernel<KS, MODE, RN>, tmQ, tmV, tmO, prm);
}

// Output rows of the off-grid leading tokens: out = q^ S / pi + 1/2 s (no convolution, no bias), from the
// final state the state kernel left in the workspace.  One block of 64 threads per (plane, token), thread =
// channel.  mode 0: 64-wide heads; 1: token pairs (width 32, the state is the sum of the two diagonal
// blocks); 2: two width-32 heads side by side (each half of the row is its own head).
__global__ void __launch_bounds__(64)
tc_prefix_rows_kernel(const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out,
                      const float* __restrict__ state, Layout lq, Layout lo, int hdiv, int prefix, int mode,
                      float eps2, int rownorm, int n_tokens) {
    __shared__ float qs[kD];
    __shared__ float part[2];
    const int plane = blockIdx.x / prefix, t = blockIdx.x % prefix, j = threadIdx.x;
    const int width = (mode == 1) ? 32 : kD;  // elements of this plane's token rows
    const __nv_bfloat16* qrow = q + plane_offset(lq, plane, hdiv) + t * lq.token;
    const float x = (j < width) ? __bfloat162float(qrow[j]) : 0.f;
    qs[j] = x;
    float ss = x * x;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((j & 31) == 0) part[j >> 5] = ss;
    __syncthreads();
    if (j >= width) return;
    const float* st = state + (size_t)plane * (kD * kD + kD + (rownorm ? kD : 0));
    const float* sk = st + kD * kD + kD;  // row-sum normalisation: sum of the unit key rows (per token parity / head)
    float nrm2, acc = 0.f, sum, qk = 0.f;
    if (mode == 0) {
        nrm2 = part[0] + part[1];
        for (int i = 0; i < kD; ++i) acc = fmaf(qs[i], st[i * kD + j], acc);
        sum = st[kD * kD + j];
        if (rownorm) for (int i = 0; i < kD; ++i) qk = fmaf(qs[i], sk[i], qk);
    } else if (mode == 1) {
        nrm2 = part[0];
        for (int i = 0; i < 32; ++i) acc = fmaf(qs[i], st[i * kD + j] + st[(32 + i) * kD + 32 + j], acc);
        sum = st[kD * kD + j] + st[kD * kD + 32 + j];
        if (rownorm) for (int i = 0; i < 32; ++i) qk = fmaf(qs[i], sk[i] + sk[32 + i], qk);
    } else {
        const int h0 = j & 32;  // first channel of this thread's head within the row
        nrm2 = part[j >> 5];
        for (int i = 0; i < 32; ++i) acc = fmaf(qs[h0 + i], st[(h0 + i) * kD + j], acc);
        sum = st[kD * kD + j];
        if (rownorm) for (int i = 0; i < 32; ++i) qk = fmaf(qs[h0 + i], sk[h0 + i], qk);
    }
    const float rq = rsqrtf(fmaxf(nrm2, eps2));
    float o = fmaf(acc * kInvPi, rq, 0.5f * sum);
    if (rownorm) o /= fmaf(qk * kInvPi, rq, 0.5f * (float)n_tokens);
    out[plane_offset(lo, plane, hdiv) + t * lo.token + j] = __float2bfloat16_rn(o);
}

}  // namespace

cudaError_t launch_prefix_rows(const Problem& p, const float* state, cudaStream_t st) {
    if (p.prefix <= 0) return cudaSuccess;
    const int mode = p.d == 32 ? 1 : (p.blockdiag ? 2 : 0);
    tc_prefix_rows_kernel<<<(unsigned)(p.BH * p.prefix), 64, 0, st>>>(
        static_cast<const __nv_bfloat16*>(p.q), static_cast<__nv_bfloat16*>(p.out), state, p.lq, p.lo, p.hdiv,
        p.prefix, mode, p.eps2, p.rownorm ? 1 : 0, p.N);
    return cudaGetLastError();
}

namespace {
template <bool RN>
cudaError_t launch_apply_rn(const Problem& p, const float* partial, int P, unsigned* status, cudaStream_t st) {
    if (p.d == 32)
        return p.ksize == 3 ? launch_apply_ks<3, 1, RN>(p, partial, P, status, st)
                            : launch_apply_ks<5, 1, RN>(p, partial, P, status, st);
    if (p.blockdiag)
        return p.ksize == 3 ? launch_apply_ks<3, 2, RN>(p, partial, P, status, st)
                            : launch_apply_ks<5, 2, RN>(p, partial, P, status, st);
    return p.ksize == 3 ? launch_apply_ks<3, 0, RN>(p, partial, P, status, st)
                        : launch_apply_ks<5, 0, RN>(p, partial, P, status, st);
}
}  // namespace

cudaError_t launch_apply(const Problem& p, const float* partial, int P, unsigned* status, cudaStream_t st) {
    return p.rownorm ? launch_apply_rn<true>(p, partial, P, status, st) : launch_apply_rn<false>(p, partial, P, status, st);
}

}  // namespace tc
}  // namespace castling

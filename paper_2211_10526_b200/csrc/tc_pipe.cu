// Whole forward pass of the tensor-core path as ONE persistent kernel (bf16; width-64 heads, or width-32
// heads packed two to a 128-byte row):
//     S = sum_n k^_n^T v_n,  s = sum_n v_n            (state, per (b,h))
//     out_t = (1/pi) q^_t S + 1/2 s + bias + DWConv(V)_t                              (Eq. 9)
// One CTA per multiprocessor, launched cooperatively so that all CTAs are resident.  Every CTA runs two
// pipelines side by side, in different warps:
//   state pipeline   warp 2 (TMA: K and V tiles of 64 rows), warp 3 (UMMAs, A = [K^ ; 1 0 0 ...] so that
//                    accumulator row 64 is the token sum of V), warps 12..15 (scale every K row by
//                    1 / max(||k||, eps) in place, read the finished accumulator out of TMEM, reduce the
//                    token splits of a plane in a fixed order, publish the plane's state and raise its flag)
//   apply pipeline   warp 0 (TMA: Q patch and V patch with halo), warp 1 (UMMAs: acc = Q S'), warps 4..11
//                    (||q||, accumulator rows scaled by 1/||q|| to shared memory as fp32), conv warps
//                    (depthwise convolution of the V patch on CUDA cores, lane = channel pair; add the
//                    scaled accumulator row, 1/2 s and the bias; one rounding to bf16; 128-byte rows stored
//                    straight to memory)
// The state pipeline walks the planes in order and never waits for the apply pipeline (except for an
// optional bound on how many planes it may run ahead); the apply pipeline of a plane waits for that
// plane's flag.  While plane p is being applied, the states of the planes after it are being built, so
// the V rows that the apply pipeline needs were read moments ago and are served from L2: V comes
// from HBM once.  Every wait is bounded; a wait that runs out raises a bit in the status word, and every
// CTA that sees the bit leaves.
#include "tc_common.cuh"
#include "tc_host.cuh"

namespace castling {
namespace tc {
namespace {

constexpr int kD = 64;
constexpr int kTY = 8, kTX = 16;            // patch: 8 rows x 16 columns of 128-byte rows
constexpr int kPatch = kTY * kTX;
constexpr int kQBytes = kPatch * kD * 2;    // 16 KiB
constexpr int kStgRow = kD * 4;             // fp32 accumulator row; 16-byte chunk c of row t sits at chunk c ^ (t & 7)
constexpr int kStgBytes = kPatch * kStgRow; // 32 KiB
constexpr int kEpiWarps = 8, kEpiThreads = kEpiWarps * 32;
constexpr int kNormWarps = 4, kNormThreads = kNormWarps * 32;
constexpr int kSTile = 64;                  // rows per state stage
constexpr int kSTileBytes = kSTile * 128;   // 8 KiB per operand tile
constexpr int kSStage = 2 * kSTileBytes;    // K then V
constexpr int kSStages = 3;
constexpr int kOnesBytes = 2048;
constexpr int kTmemCols = 256;              // [0,128): two apply accumulators; [128,256): two state accumulators
constexpr int kGroup = 4;                   // splits per first-level reduction group
constexpr int kWords = kD * kD + kD;        // one state: S then s
constexpr int kFirstWarpEpi = 4, kFirstWarpNorm = kFirstWarpEpi + kEpiWarps, kFirstWarpConv = kFirstWarpNorm + kNormWarps;
constexpr unsigned kBit = kStatusPipeTimeout;

template <int KS, bool PAIR> struct PGeo {
    static constexpr int kConvRows = (KS == 3) ? 2 : 4;
    static constexpr int kConvWarps = 2 * kTY / kConvRows, kConvThreads = kConvWarps * 32;
    static constexpr int kThreads = 32 * kFirstWarpConv + kConvThreads;
    static constexpr int R = KS / 2;
    static constexpr int HC = PAIR ? (R + 1) / 2 : R;   // halo columns on each side
    static constexpr int HY = kTY + 2 * R, HX = kTX + 2 * HC;
    static constexpr int kVBytes = HY * HX * kD * 2;
    static constexpr int kStage = ((kQBytes + kVBytes + 1023) / 1024) * 1024;
    static constexpr int kStages = (KS == 3) ? 3 : 2;
    // 3x3: one staging buffer, the conv warps hold the first half of a patch's results in registers
    // while the epilogue warps fill it; 5x5 (larger window in registers): two staging buffers
    static constexpr int kStgBufs = (KS == 3) ? 1 : 2;
    static constexpr int kHold = (kStgBufs == 1) ? kTX / 4 : 0;   // output columns per warp held back
    static constexpr int kOffS = 0, kOffStg = 8192, kOffStages = kOffStg + kStgBufs * kStgBytes;
    static constexpr int kOffSStages = kOffStages + kStages * kStage;
    static constexpr int kOffOnes = kOffSStages + kSStages * kSStage;
    static constexpr int kOffRq = kOffOnes + kOnesBytes;          // [2][2][kPatch] partial sums of squares
    static constexpr int kOffBar = kOffRq + 2 * 2 * kPatch * 4;
    static constexpr size_t kSmem = 1024 + kOffBar + 512;
};

struct PipeParams {
    float* partial;                // [BH][P][kWords] per-split sums (P > 1)
    float* state;                  // [BH][kWords] final sums
    unsigned* ctr;                 // kPipeCtrHeader words, then kPipeCtrPerPlane per plane; all zero between calls
    const __nv_bfloat16* w;        // [H*d][KS][KS]
    const __nv_bfloat16* bias;     // [H*d] or nullptr
    __nv_bfloat16* out;            // first grid token of plane 0
    Layout lo;
    int flat;                      // the planes have one uniform stride: the apply tensor maps are 4-D
    int H, head0, BH, hdiv;
    int tilesX, tilesY;            // patches per plane
    int gridH, cols;               // grid rows; 128-byte columns per grid row
    int s_tiles, s_per, P;         // state tiles per plane, tiles per split, splits per plane
    int plane_order;               // every CTA takes a share of every plane, plane after plane (long sequences)
    int ahead;                     // the state pipeline starts plane p only when plane p - ahead is applied
    float eps2;
    unsigned* status;
};

// This CTA's patches, in the order every role of the apply pipeline visits them.
struct PatchWalk {
    int bh, rem, end, left, tpb, G, cta, BH;
    bool by_plane;
    __device__ void init(const PipeParams& prm) {
        tpb = prm.tilesX * prm.tilesY; G = (int)gridDim.x; cta = (int)blockIdx.x; BH = prm.BH;
        by_plane = prm.plane_order != 0;
        if (!by_plane) {  // one contiguous range of the plane-major patch list
            const long long n = (long long)BH * tpb;
            const int g0 = (int)(n * cta / G), g1 = (int)(n * (cta + 1) / G);
            left = g1 - g0; bh = g0 / tpb; rem = g0 - bh * tpb; end = tpb;
        } else {
            bh = -1; rem = end = 0; left = 1;
            next_plane();
        }
    }
    __device__ void next_plane() {
        while (true) {
            if (++bh >= BH) { left = 0; return; }
            const int cc = (cta + 37 * bh) % G;  // the larger shares rotate over the CTAs from plane to plane
            rem = (int)((long long)tpb * cc / G); end = (int)((long long)tpb * (cc + 1) / G);
            if (rem < end) return;
        }
    }
    __device__ bool valid() const { return left > 0; }
    __device__ void step() {
        ++rem;
        if (!by_plane) { --left; if (rem == tpb) { rem = 0; ++bh; } }
        else if (rem == end) next_plane();
    }
};

// Bounded wait for a counter in global memory to reach `want`.  Gives up (returns false) when the limit
// runs out (raising the status bit), when this CTA has given up elsewhere, or when any CTA has raised a bit.
__device__ __forceinline__ bool wait_counter(const unsigned* p, unsigned want, volatile int* abort_flag, unsigned* status) {
    auto poll = [&]() { unsigned v; asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v; };
    if (poll() >= want) return true;
    const unsigned long long t0 = global_ns();
    uint32_t spins = 0;
    while (true) {
        __nanosleep(100);
        if (poll() >= want) return true;
        if ((++spins & 63u) == 0) {
            if (*abort_flag) return false;
            if (*reinterpret_cast<volatile unsigned*>(status) != 0) { *abort_flag = 1; return false; }
            if (global_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; atomicOr(status, kBit); return false; }
        }
    }
}

// Named barrier over `threads` threads that also tells every one of them whether any of them has failed.
__device__ __forceinline__ bool barrier_any(uint32_t id, uint32_t threads, bool failed) {
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %3, 0;\n\t"
                 "barrier.cta.red.or.pred q, %1, %2, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(r) : "r"(id), "r"(threads), "r"((uint32_t)failed) : "memory");
    return r != 0;
}

__device__ __forceinline__ void st_global_hint(void* p, uint32_t v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.b32 [%0], %1, %2;" ::"l"(p), "r"(v), "l"(policy) : "memory");
}

// Sum `n` states of kWords floats, `stride` floats apart, in index order into dst (128 threads).
__device__ __forceinline__ void sum_states(const float* src, size_t stride, int n, float* dst, int t) {
    constexpr int kWords4 = kWords / 4;
    for (int i = t; i < kWords4; i += kNormThreads) {
        float4 acc = __ldcg(reinterpret_cast<const float4*>(src) + i);
        int m = 1;
        for (; m + 3 <= n; m += 3) {
            const float4 a = __ldcg(reinterpret_cast<const float4*>(src + (size_t)m * stride) + i);
            const float4 b = __ldcg(reinterpret_cast<const float4*>(src + (size_t)(m + 1) * stride) + i);
            const float4 c = __ldcg(reinterpret_cast<const float4*>(src + (size_t)(m + 2) * stride) + i);
            acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
            acc.x += b.x; acc.y += b.y; acc.z += b.z; acc.w += b.w;
            acc.x += c.x; acc.y += c.y; acc.z += c.z; acc.w += c.w;
        }
        for (; m < n; ++m) {
            const float4 a = __ldcg(reinterpret_cast<const float4*>(src + (size_t)m * stride) + i);
            acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
        }
        reinterpret_cast<float4*>(dst)[i] = acc;
    }
}

// MODE 0: width-64 heads; 1: width-32 heads, two adjacent tokens per 128-byte row; 2: two width-32 heads side
// by side in one row (block-diagonal state).
template <int KS, int MODE>
__global__ void __launch_bounds__((PGeo<KS, MODE == 1>::kThreads), 1)
tc_pipe_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmVs,
               const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmVh,
               const PipeParams prm) {
    constexpr bool PAIR = (MODE == 1), BLOCKDIAG = (MODE == 2), HALVES = PAIR || BLOCKDIAG;
    using G = PGeo<KS, PAIR>;
    constexpr int NA = G::kStages, NS = kSStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* S_s = smem + G::kOffS;
    uint8_t* stg = smem + G::kOffStg;
    uint8_t* stages = smem + G::kOffStages;
    uint8_t* sstages = smem + G::kOffSStages;
    uint8_t* ones = smem + G::kOffOnes;
    float* rq_s = reinterpret_cast<float*>(smem + G::kOffRq);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + G::kOffBar);
    uint64_t* a_full = bars;                 // [NA] Q and V patch landed
    uint64_t* a_empty = a_full + NA;         // [NA] stage consumed (conv + epilogue warps, UMMA commit)
    uint64_t* acc_full = a_empty + NA;       // [2]  apply UMMAs retired
    uint64_t* acc_free = acc_full + 2;       // [2]  accumulator read out (epilogue threads)
    uint64_t* stg_full = acc_free + 2;       // [2]  staging written (epilogue threads)
    uint64_t* stg_free = stg_full + 2;       // [2]  staging read (conv threads)
    uint64_t* s_ready = stg_free + 2;        //      S' of the current plane written (epilogue threads)
    uint64_t* s_full = s_ready + 1;          // [NS] K and V tile landed
    uint64_t* s_scaled = s_full + NS;        // [NS] K rows normalised
    uint64_t* s_empty = s_scaled + NS;       // [NS] state UMMAs of the stage retired
    uint64_t* sacc_full = s_empty + NS;      // [2]  accumulation of an item retired
    uint64_t* sacc_free = sacc_full + 2;     // [2]  accumulator read out
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sacc_free + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* last_slot = reinterpret_cast<int*>(tmem_slot + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_cta = (int)gridDim.x, cta = (int)blockIdx.x;
    const int n_items = prm.BH * prm.P;
    unsigned* plane_ctr = prm.ctr + kPipeCtrHeader;

    if (tid == 0) {
        for (int s = 0; s < NA; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], G::kConvThreads + kEpiThreads + 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1); mbar_init(&acc_free[b], kEpiThreads);
            mbar_init(&stg_full[b], kEpiThreads); mbar_init(&stg_free[b], G::kConvThreads);
            mbar_init(&sacc_full[b], 1); mbar_init(&sacc_free[b], kNormThreads);
        }
        mbar_init(s_ready, kEpiThreads);
        for (int s = 0; s < NS; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_scaled[s], kNormThreads); mbar_init(&s_empty[s], 1); }
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmVs); tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmVh);
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    if (warp >= kFirstWarpNorm && warp < kFirstWarpConv) {
        // constant block of the state A operand: for each of 16 token rows, element 64 (first of the second
        // 64-wide block along M) is 1.0 and the rest 0; 16-byte chunk c of row r sits at chunk c ^ (r & 7)
        const int t = tid - 32 * kFirstWarpNorm, r = t >> 3, c = t & 7;
        uint4 val = make_uint4(0, 0, 0, 0);
        if ((c ^ (r & 7)) == 0) val.x = 0x3f80u;
        *reinterpret_cast<uint4*>(ones + r * 128 + c * 16) = val;
        fence_proxy_async_smem();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tmem_state = tmem + 128;

    if (warp == 0) {
        // ================= apply pipeline: TMA producer =================
        if (lane == 0) {
            int issued = 0;
            const uint64_t pol_q = l2_policy_evict_first();  // Q is read once
            PatchWalk wk; wk.init(prm);
            for (int it = 0; wk.valid(); ++it, wk.step()) {
                const int s = it % NA, use = it / NA;
                if (use > 0 && !mbar_wait(&a_empty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) break;
                const int y0 = (wk.rem / prm.tilesX) * kTY, x0 = (wk.rem % prm.tilesX) * kTX;
                uint8_t* qs = stages + s * G::kStage;
                mbar_expect_tx(&a_full[s], kQBytes + G::kVBytes);
                if (prm.flat) {
                    tma_load_4d_hint(qs, &tmQ, &a_full[s], 0, x0, y0, wk.bh, pol_q);
                    tma_load_4d(qs + kQBytes, &tmVh, &a_full[s], 0, x0 - G::HC, y0 - G::R, wk.bh);
                } else {
                    const int pb = wk.bh / prm.hdiv, ph = wk.bh - pb * prm.hdiv;
                    tma_load_5d_hint(qs, &tmQ, &a_full[s], 0, x0, y0, ph, pb, pol_q);
                    tma_load_5d(qs + kQBytes, &tmVh, &a_full[s], 0, x0 - G::HC, y0 - G::R, ph, pb);
                }
                ++issued;
            }
            if (*abort_flag) {  // giving up: let copies already in flight land before shared memory goes away
                for (int i = max(0, issued - NA); i < issued; ++i)
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&a_full[i % NA], (i / NA) & 1); ++spin) {}
            }
        }
    } else if (warp == 1) {
        // ================= apply pipeline: UMMA issuer =================
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, kD, false, true);
            const uint32_t s_addr = smem_u32(S_s);
            int prev_bh = -1, seg = 0;
            PatchWalk wk; wk.init(prm);
            for (int it = 0; wk.valid(); ++it, wk.step()) {
                const int s = it % NA, use = it / NA, b = it & 1, ub = it >> 1;
                if (wk.bh != prev_bh) {
                    if (!mbar_wait(s_ready, seg & 1, abort_flag, prm.status, kBit)) break;
                    ++seg; prev_bh = wk.bh;
                }
                if (!mbar_wait(&a_full[s], use & 1, abort_flag, prm.status, kBit)) break;
                if (ub > 0 && !mbar_wait(&acc_free[b], (ub - 1) & 1, abort_flag, prm.status, kBit)) break;
                tcgen05_fence_after_sync();
                const uint32_t q_addr = smem_u32(stages + s * G::kStage);
#pragma unroll
                for (int k = 0; k < kD / 16; ++k) {
                    const uint64_t a = umma_desc_sw128(q_addr + k * 32, 0, 1024);        // K-major rows of 128 B
                    const uint64_t bd = umma_desc_sw128(s_addr + k * 2048, 0, 1024);     // N-major, 16 K-rows per step
                    umma_bf16(tmem + b * kD, a, bd, idesc, k != 0);
                }
                umma_commit(&acc_full[b]);
                umma_commit(&a_empty[s]);  // the same UMMAs have finished reading the Q patch
            }
        }
    } else if (warp == 2) {
        // ================= state pipeline: TMA producer =================
        if (lane == 0) {
            int issued = 0;
            // K is read once; V is read again by the apply pipeline: keep it in L2 as long as possible
            const uint64_t pol_k = l2_policy_evict_first(), pol_v = l2_policy_evict_last();
            const unsigned applied = (unsigned)(prm.tilesX * prm.tilesY * G::kConvWarps);  // arrivals of a whole plane
            bool ok = true;
            for (int item = cta; item < n_items && ok; item += n_cta) {
                const int plane = item / prm.P, part = item - plane * prm.P;
                const int t0 = part * prm.s_per, t1 = min(prm.s_tiles, t0 + prm.s_per);
                if (plane >= prm.ahead &&
                    !wait_counter(plane_ctr + (size_t)(plane - prm.ahead) * kPipeCtrPerPlane + kPipeCtrApplied, applied,
                                  abort_flag, prm.status)) break;
                const int pb = plane / prm.hdiv, ph = plane - pb * prm.hdiv;
                for (int t = t0; t < t1; ++t, ++issued) {
                    const int s = issued % NS, use = issued / NS;
                    if (use > 0 && !mbar_wait(&s_empty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) { ok = false; break; }
                    uint8_t* ks = sstages + s * kSStage;
                    mbar_expect_tx(&s_full[s], kSStage);
                    tma_load_4d_hint(ks, &tmK, &s_full[s], 0, t * kSTile, ph, pb, pol_k);
                    tma_load_4d_hint(ks + kSTileBytes, &tmVs, &s_full[s], 0, t * kSTile, ph, pb, pol_v);
                }
            }
            if (*abort_flag) {
                for (int i = max(0, issued - NS); i < issued; ++i)
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&s_full[i % NS], (i / NS) & 1); ++spin) {}
            }
        }
    } else if (warp == 3) {
        // ================= state pipeline: UMMA issuer =================
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, kD, true, true);
            const uint32_t ones_addr = smem_u32(ones);
            bool ok = true;
            int gt = 0, k_item = 0;  // tiles and items issued so far
            for (int item = cta; item < n_items && ok; item += n_cta, ++k_item) {
                const int plane = item / prm.P, part = item - plane * prm.P;
                const int t0 = part * prm.s_per, t1 = min(prm.s_tiles, t0 + prm.s_per);
                const int buf = k_item & 1;
                if (k_item >= 2) ok = mbar_wait(&sacc_free[buf], ((k_item >> 1) - 1) & 1, abort_flag, prm.status, kBit);
                for (int t = t0; t < t1 && ok; ++t, ++gt) {
                    const int s = gt % NS, use = gt / NS;
                    ok = mbar_wait(&s_scaled[s], use & 1, abort_flag, prm.status, kBit);
                    if (!ok) break;
                    tcgen05_fence_after_sync();
                    const uint32_t ka = smem_u32(sstages + s * kSStage), va = ka + kSTileBytes;
#pragma unroll
                    for (int j = 0; j < kSTile / 16; ++j) {  // one UMMA per 16 rows (K = 16)
                        const uint32_t a0 = ka + j * 2048, b0 = va + j * 2048;
                        umma_bf16(tmem_state + buf * kD, umma_desc_sw128(a0, ones_addr - a0, 1024),
                                  umma_desc_sw128(b0, 0, 1024), idesc, (t != t0) || (j != 0));
                    }
                    umma_commit(&s_empty[s]);
                }
                if (ok) umma_commit(&sacc_full[buf]);
            }
        }
    } else if (warp < kFirstWarpNorm) {
        // ================= apply pipeline: epilogue, thread = (token row of the patch, half of the channels) =================
        const int quarter = warp & 3, row = quarter * 32 + lane, et = tid - 32 * kFirstWarpEpi;
        const int half = (warp - kFirstWarpEpi) >> 2;  // channels half*32 .. half*32 + 31
        int prev_bh = -1;
        bool failed = false;
        PatchWalk wk; wk.init(prm);
        for (int it = 0; wk.valid(); ++it, wk.step()) {
            const int b = it & 1, ub = it >> 1, s = it % NA, use = it / NA;
            const int sb = (G::kStgBufs == 2) ? b : 0, su = (G::kStgBufs == 2) ? ub : it;  // staging buffer and its use count
            if (wk.bh != prev_bh && !failed) {
                prev_bh = wk.bh;
                // every UMMA that read the previous S' has retired (its acc_full was waited on below)
                bool ready = true;
                if (lane == 0)
                    ready = wait_counter(plane_ctr + (size_t)wk.bh * kPipeCtrPerPlane + kPipeCtrReady, 1u, abort_flag, prm.status);
                ready = __shfl_sync(0xffffffffu, (int)ready, 0) != 0;
                if (!ready) { failed = true; }
                else {
                    const int i = et >> 2, part = et & 3;  // row i of the operand, 16 columns part*16 ..
                    const float* st = prm.state + (size_t)wk.bh * kWords;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        float4 lo, hi;
                        if (!PAIR) {
                            const float4* src = reinterpret_cast<const float4*>(st + i * kD + part * 16);
                            lo = __ldcg(src + 2 * c); hi = __ldcg(src + 2 * c + 1);
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
                                const float4 l0 = __ldcg(s0), h0 = __ldcg(s0 + 1), l1 = __ldcg(s1), h1 = __ldcg(s1 + 1);
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
                    }
                    fence_proxy_async_smem();
                    mbar_arrive(s_ready);
                }
            }
            float a[32];
            if (!failed) {
                // this thread's half of sum(q^2) for its token; the other half comes from the partner warp
                failed = __any_sync(0xffffffffu, !mbar_wait(&a_full[s], use & 1, abort_flag, prm.status, kBit));
            }
            if (!failed) {
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
                rq_s[(b * 2 + half) * kPatch + row] = (ss[0] + ss[1]) + (ss[2] + ss[3]);
                mbar_arrive(&a_empty[s]);  // the Q rows of this stage have been read
                failed = __any_sync(0xffffffffu, !mbar_wait(&acc_full[b], ub & 1, abort_flag, prm.status, kBit));
            }
            if (!failed) {
                tcgen05_fence_after_sync();
                float a0[16], a1[16];
                tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + b * kD + half * 32, a0);
                tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + b * kD + half * 32 + 16, a1);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 16; ++e) { a[e] = a0[e]; a[16 + e] = a1[e]; }
                tcgen05_fence_before_sync();
                mbar_arrive(&acc_free[b]);
            }
            if (!HALVES) {
                // both halves of every row's sum of squares become visible; every thread learns whether one gave up
                if (barrier_any(1, kEpiThreads, failed)) break;
            } else if (failed) break;
            const float rq = HALVES ? rsqrtf(fmaxf(rq_s[(b * 2 + half) * kPatch + row], prm.eps2))   // half row = one token / one head
                                    : rsqrtf(fmaxf(rq_s[(b * 2) * kPatch + row] + rq_s[(b * 2 + 1) * kPatch + row], prm.eps2));
            // the conv warps have read the previous contents of this staging buffer
            if (su > 0 && __any_sync(0xffffffffu, !mbar_wait(&stg_free[sb], (su - 1) & 1, abort_flag, prm.status, kBit))) {
                if (!HALVES) { failed = true; continue; }   // leave together at the next barrier
                break;
            }
            uint8_t* srow = stg + sb * kStgBytes + row * kStgRow;
#pragma unroll
            for (int e = 0; e < 8; ++e)
                *reinterpret_cast<float4*>(srow + (((half * 8 + e) ^ (row & 7)) << 4)) =
                    make_float4(a[4 * e] * rq, a[4 * e + 1] * rq, a[4 * e + 2] * rq, a[4 * e + 3] * rq);
            mbar_arrive(&stg_full[sb]);
        }
    } else if (warp < kFirstWarpConv) {
        // ================= state pipeline: K normalisation, accumulator read-out, split reduction =================
        const int t = tid - 32 * kFirstWarpNorm;   // 0..127: row t >> 1 of the stage, half t & 1 of that row
        const int quarter = warp & 3;
        const int r = t >> 1, hf = t & 1;
        bool ok = true;
        // read the finished accumulator of the k-th item of this CTA out of TMEM: rows 0..63 are S, row 64 is s
        auto flush = [&](int k_item, float* dst) -> bool {
            const int buf = k_item & 1;
            if (!mbar_wait(&sacc_full[buf], (k_item >> 1) & 1, abort_flag, prm.status, kBit)) return false;
            tcgen05_fence_after_sync();
            if (quarter < 3) {
                const int row = quarter * 32 + lane;
#pragma unroll
                for (int cc = 0; cc < kD / 16; ++cc) {
                    float v[16];
                    tmem_ld16(tmem_state + ((uint32_t)(quarter * 32) << 16) + buf * kD + cc * 16, v);
                    tmem_ld_wait();
                    if (row <= kD) {
                        float4* o4 = reinterpret_cast<float4*>(dst + row * kD + cc * 16);  // row 64 lands on s
#pragma unroll
                        for (int e = 0; e < 4; ++e) o4[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                    }
                }
            }
            tcgen05_fence_before_sync();
            mbar_arrive(&sacc_free[buf]);
            return true;
        };
        // After an item's partial state is in memory: count it; the last split of a group sums the group, the
        // last group sums the groups (both in index order: the result does not depend on who came last), writes
        // the plane's state and raises its flag.  With one split per plane the state is already final.
        auto publish = [&](int item) {
            const int plane = item / prm.P, part = item - plane * prm.P;
            unsigned* pc = plane_ctr + (size_t)plane * kPipeCtrPerPlane;
            __threadfence();
            named_barrier_sync(2, kNormThreads);
            if (prm.P > 1) {
                const int n_groups = (prm.P + kGroup - 1) / kGroup, grp = part / kGroup;
                const int first = grp * kGroup, members = min(kGroup, prm.P - first);
                float* base = prm.partial + (size_t)plane * prm.P * kWords;
                if (t == 0) *last_slot = (atomicAdd(&pc[grp], 1u) == (unsigned)(members - 1));
                named_barrier_sync(2, kNormThreads);
                const bool last_in_group = *last_slot != 0;
                named_barrier_sync(2, kNormThreads);
                if (!last_in_group) return;
                __threadfence();
                if (members > 1) sum_states(base + (size_t)first * kWords, kWords, members, base + (size_t)first * kWords, t);
                __threadfence();
                named_barrier_sync(2, kNormThreads);
                if (t == 0) { pc[grp] = 0; *last_slot = (atomicAdd(&pc[kPipeCtrGroups], 1u) == (unsigned)(n_groups - 1)); }
                named_barrier_sync(2, kNormThreads);
                const bool last_group = *last_slot != 0;
                named_barrier_sync(2, kNormThreads);
                if (!last_group) return;
                __threadfence();
                sum_states(base, (size_t)kGroup * kWords, n_groups, prm.state + (size_t)plane * kWords, t);
                __threadfence();
                named_barrier_sync(2, kNormThreads);
                if (t == 0) pc[kPipeCtrGroups] = 0;
            }
            if (t == 0) {
                __threadfence();
                asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(pc + kPipeCtrReady), "r"(1u) : "memory");
            }
        };
        auto item_dst = [&](int item) -> float* {
            return prm.P > 1 ? prm.partial + (size_t)item * kWords : prm.state + (size_t)item * kWords;  // item = plane * P + part
        };
        int gt = 0, k_item = 0, prev_item = -1;
        bool dead = false;  // some thread of the group gave up: everybody leaves (decided at a barrier, so together)
        for (int item = cta; item < n_items; item += n_cta, ++k_item) {
            const int plane = item / prm.P, part = item - plane * prm.P;
            const int t0 = part * prm.s_per, t1 = min(prm.s_tiles, t0 + prm.s_per);
            for (int tt = t0; tt < t1 && ok; ++tt, ++gt) {
                const int s = gt % NS, use = gt / NS;
                ok = mbar_wait(&s_full[s], use & 1, abort_flag, prm.status, kBit);
                if (!ok) break;
                uint8_t* rowp = sstages + s * kSStage + r * 128;
                uint4 c[4];
                float ss = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    c[j] = *reinterpret_cast<const uint4*>(rowp + (((4 * hf + j) ^ (r & 7)) << 4));
                    const uint32_t w4[4] = {c[j].x, c[j].y, c[j].z, c[j].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float lo = bf16lo(w4[e]), hi = bf16hi(w4[e]);
                        ss = fmaf(lo, lo, ss); ss = fmaf(hi, hi, ss);
                    }
                }
                if (!HALVES) ss += __shfl_xor_sync(0xffffffffu, ss, 1);  // the two halves of a row sit in neighbouring lanes
                const float rk = 1.0f / sqrtf(fmaxf(ss, prm.eps2));
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint4 o;
                    o.x = pack_bf16x2(bf16lo(c[j].x) * rk, bf16hi(c[j].x) * rk);
                    o.y = pack_bf16x2(bf16lo(c[j].y) * rk, bf16hi(c[j].y) * rk);
                    o.z = pack_bf16x2(bf16lo(c[j].z) * rk, bf16hi(c[j].z) * rk);
                    o.w = pack_bf16x2(bf16lo(c[j].w) * rk, bf16hi(c[j].w) * rk);
                    *reinterpret_cast<uint4*>(rowp + (((4 * hf + j) ^ (r & 7)) << 4)) = o;
                }
                fence_proxy_async_smem();
                mbar_arrive(&s_scaled[s]);
            }
            // the previous item is read out one item late, so that its UMMAs overlap this item's normalisation
            if (prev_item >= 0 && ok) ok = flush(k_item - 1, item_dst(prev_item));
            if (barrier_any(3, kNormThreads, !ok)) { dead = true; break; }
            if (prev_item >= 0) publish(prev_item);
            prev_item = item;
        }
        if (!dead && prev_item >= 0) {
            ok = flush(k_item - 1, item_dst(prev_item));
            if (!barrier_any(3, kNormThreads, !ok)) publish(prev_item);
        }
    } else {
        // ================= apply pipeline: depthwise convolution + combine + store =================
        const int cwi = warp - kFirstWarpConv;
        const int cw = cwi >> 1, xh = cwi & 1;  // row group and column half of the patch
        constexpr int kCX = kTX / 2;
        constexpr int R = G::R, RO = G::kConvRows, ROWS = RO + 2 * R, HOLD = G::kHold;
        float2 wreg[KS][KS];
        float2 cinit = make_float2(0.f, 0.f);
        int prev_bh = -1;
        const uint64_t pol_o = l2_policy_evict_first();  // the output is not read back here
        const long long row_stride = PAIR ? kD : prm.lo.token;  // elements between 128-byte rows of the output
        PatchWalk wk; wk.init(prm);
        for (int it = 0; wk.valid(); ++it, wk.step()) {
            const int s = it % NA, use = it / NA, b = it & 1, ub = it >> 1;
            const int sb = (G::kStgBufs == 2) ? b : 0, su = (G::kStgBufs == 2) ? ub : it;
            const int bh = wk.bh;
            if (bh != prev_bh) {
                prev_bh = bh;
                bool ready = true;
                if (lane == 0)
                    ready = wait_counter(plane_ctr + (size_t)bh * kPipeCtrPerPlane + kPipeCtrReady, 1u, abort_flag, prm.status);
                if (!__shfl_sync(0xffffffffu, (int)ready, 0)) break;
                // this lane's channel pair: 2*lane of 64 channels, or (PAIR) 2*(lane & 15) of 32 channels
                // for the token of parity lane >> 4
                const int cp2 = PAIR ? 2 * (lane & 15) : 2 * lane;
                const int ch = ((prm.head0 + bh) % prm.H) * (PAIR ? 32 : kD) + cp2;
                const float* sv = prm.state + (size_t)bh * kWords + kD * kD;
                float s0, s1;
                if (PAIR) {  // token sum = sum of the two halves of the paired sums
                    s0 = __ldcg(sv + cp2) + __ldcg(sv + 32 + cp2);
                    s1 = __ldcg(sv + cp2 + 1) + __ldcg(sv + 32 + cp2 + 1);
                } else {
                    s0 = __ldcg(sv + cp2); s1 = __ldcg(sv + cp2 + 1);
                }
                cinit.x = 0.5f * s0; cinit.y = 0.5f * s1;
                if (prm.bias) { cinit.x += __bfloat162float(prm.bias[ch]); cinit.y += __bfloat162float(prm.bias[ch + 1]); }
#pragma unroll
                for (int dy = 0; dy < KS; ++dy)
#pragma unroll
                    for (int dx = 0; dx < KS; ++dx)
                        wreg[dy][dx] = make_float2(__bfloat162float(prm.w[(size_t)ch * KS * KS + dy * KS + dx]),
                                                   __bfloat162float(prm.w[(size_t)(ch + 1) * KS * KS + dy * KS + dx]));
            }
            if (__any_sync(0xffffffffu, !mbar_wait(&a_full[s], use & 1, abort_flag, prm.status, kBit))) break;
            // Window of KS tokens per halo row, sliding along x.  Token t (relative to the first token this
            // lane needs) sits U bytes after token t-1: U = 128, one token per column, or (PAIR) 64.
            // One output column advances the window by STEP tokens (2 when PAIR: the lane's token keeps
            // its parity).  Slot of token t in the rotating window: t % KS (t is a compile-time value).
            constexpr int U = PAIR ? 64 : 128, STEP = PAIR ? 2 : 1;
            const int tok0 = PAIR ? 2 * (xh * kCX + G::HC) + (lane >> 4) - R : xh * kCX;
            const uint8_t* vh = stages + s * G::kStage + kQBytes + (RO * cw) * G::HX * 128 + tok0 * U +
                                (PAIR ? (lane & 15) * 4 : lane * 4);
            const int y0 = (wk.rem / prm.tilesX) * kTY + RO * cw, x0 = (wk.rem % prm.tilesX) * kTX + xh * kCX;
            // lane's 32-bit word of the output row of patch token (RO*cw, xh*kCX)
            uint32_t* orow = reinterpret_cast<uint32_t*>(prm.out + plane_offset(prm.lo, bh, prm.hdiv) +
                                                         ((long long)y0 * prm.cols + x0) * row_stride) + lane;
            const uint8_t* srow = stg + sb * kStgBytes + ((RO * cw) * kTX + xh * kCX) * kStgRow + (lane & 1) * 8;
            const int sc = lane >> 1;
            auto combine = [&](int r, int x, float2 acc) {
                const int t = (RO * cw + r) * kTX + xh * kCX + x;
                const float2 a2 = *reinterpret_cast<const float2*>(srow + (r * kTX + x) * kStgRow + ((sc ^ (t & 7)) << 4));
                if (y0 + r < prm.gridH && x0 + x < prm.cols)
                    st_global_hint(orow + ((long long)r * prm.cols + x) * (row_stride / 2), pack_bf16x2(a2.x + acc.x, a2.y + acc.y), pol_o);
            };
            float2 win[ROWS][KS];
#pragma unroll
            for (int t = 0; t < KS - STEP; ++t)
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    const uint32_t wv = *reinterpret_cast<const uint32_t*>(vh + r * G::HX * 128 + t * U);
                    win[r][t % KS] = make_float2(bf16lo(wv), bf16hi(wv));
                }
            float2 held[HOLD > 0 ? HOLD : 1][RO];
            bool ok = true;
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
                if (x < HOLD) {
#pragma unroll
                    for (int r = 0; r < RO; ++r) held[x][r] = acc[r];
                } else {
                    if (x == HOLD) {  // the scaled accumulator rows of this patch are in the staging buffer
                        ok = !__any_sync(0xffffffffu, !mbar_wait(&stg_full[sb], su & 1, abort_flag, prm.status, kBit));
                        if (ok) {
#pragma unroll
                            for (int xx = 0; xx < HOLD; ++xx)
#pragma unroll
                                for (int r = 0; r < RO; ++r) combine(r, xx, held[xx][r]);
                        }
                    }
                    if (ok) {
#pragma unroll
                        for (int r = 0; r < RO; ++r) combine(r, x, acc[r]);
                    }
                }
            }
            if (!ok) break;
            mbar_arrive(&a_empty[s]);      // the V patch of this stage is no longer needed
            mbar_arrive(&stg_free[sb]);    // nor the staging buffer
            if (lane == 0) atomicAdd(plane_ctr + (size_t)bh * kPipeCtrPerPlane + kPipeCtrApplied, 1u);
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    // The CTA that leaves last puts the per-plane flags and counters back to zero for the next call.
    if (tid == 0) {
        __threadfence();
        *last_slot = (atomicAdd(prm.ctr, 1u) == (unsigned)(n_cta - 1));
    }
    __syncthreads();
    if (*last_slot) {
        __threadfence();
        for (int i = tid; i < prm.BH; i += blockDim.x) {
            plane_ctr[(size_t)i * kPipeCtrPerPlane + kPipeCtrReady] = 0;
            plane_ctr[(size_t)i * kPipeCtrPerPlane + kPipeCtrApplied] = 0;
        }
        if (tid == 0) prm.ctr[0] = 0;
    }
}

template <int KS, int MODE>
cudaError_t launch_pipe_ks(const Problem& p, float* partial, float* state, unsigned* ctr, unsigned* status, cudaStream_t st) {
    constexpr bool PAIR = (MODE == 1);
    using G = PGeo<KS, PAIR>;
    const bool pair = PAIR;
    const int rows = pair ? p.N / 2 : p.N;            // 128-byte rows per plane (leading off-grid tokens included)
    const int cols = pair ? p.gridW / 2 : p.gridW;    // 128-byte columns per grid row
    const uint64_t nb = (uint64_t)(p.BH / p.hdiv);
    CUtensorMap tmK, tmVs, tmQ, tmVh;
    {   // state: [64, rows, planes per batch step, batch steps]
        const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)rows, (uint64_t)p.hdiv, nb};
        const uint32_t box[4] = {kD, kSTile, 1, 1};
        const uint64_t sk[3] = {(uint64_t)(pair ? kD : p.lk.token), (uint64_t)p.lk.head,
                                (uint64_t)(nb > 1 ? p.lk.batch : p.lk.head * p.hdiv)};
        const uint64_t sv[3] = {(uint64_t)(pair ? kD : p.lv.token), (uint64_t)p.lv.head,
                                (uint64_t)(nb > 1 ? p.lv.batch : p.lv.head * p.hdiv)};
        if (!make_tensor_map_bf16(&tmK, p.k, 4, dims, sk, box, true) || !make_tensor_map_bf16(&tmVs, p.v, 4, dims, sv, box, true))
            return cudaErrorNotSupported;
    }
    const int rank = nb > 1 ? 5 : 4;
    {   // apply: [64, columns, grid rows, planes per batch step, batch steps]; the grid starts after the leading tokens
        const uint64_t dims[5] = {(uint64_t)kD, (uint64_t)cols, (uint64_t)p.gridH, (uint64_t)p.hdiv, nb};
        const uint32_t box[5] = {kD, kTX, kTY, 1, 1};
        const uint32_t boxv[5] = {kD, (uint32_t)G::HX, (uint32_t)G::HY, 1, 1};
        auto strides = [&](const Layout& l, uint64_t (&s)[4]) {
            s[0] = (uint64_t)(pair ? kD : l.token);
            s[1] = (uint64_t)(l.token * p.gridW);
            s[2] = (uint64_t)l.head;
            s[3] = (uint64_t)(nb > 1 ? l.batch : l.head * p.hdiv);
        };
        uint64_t sq[4], sv[4];
        strides(p.lq, sq); strides(p.lv, sv);
        const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + p.prefix * p.lq.token;
        const __nv_bfloat16* vg = static_cast<const __nv_bfloat16*>(p.v) + p.prefix * p.lv.token;
        if (!make_tensor_map_bf16(&tmQ, qg, rank, dims, sq, box, true) || !make_tensor_map_bf16(&tmVh, vg, rank, dims, sv, boxv, false))
            return cudaErrorNotSupported;
    }
    PipeParams prm;
    prm.partial = partial; prm.state = state; prm.ctr = ctr;
    prm.w = static_cast<const __nv_bfloat16*>(p.w);
    prm.bias = static_cast<const __nv_bfloat16*>(p.bias);
    prm.out = static_cast<__nv_bfloat16*>(p.out) + p.prefix * p.lo.token;
    prm.lo = p.lo;
    prm.flat = (rank == 4) ? 1 : 0;
    prm.H = p.H; prm.head0 = p.head0; prm.BH = p.BH; prm.hdiv = p.hdiv;
    prm.tilesX = (cols + kTX - 1) / kTX; prm.tilesY = (p.gridH + kTY - 1) / kTY;
    prm.gridH = p.gridH; prm.cols = cols;
    const PipePlan plan = plan_pipe(p.BH, rows, cols, p.gridH);
    prm.s_tiles = plan.s_tiles; prm.s_per = plan.s_per; prm.P = plan.P;
    prm.plane_order = plan.plane_order; prm.ahead = plan.ahead;
    prm.eps2 = p.eps2; prm.status = status;
    static PerDevice opt_in;  // one per instantiation
    {
        const cudaError_t e = opt_in_smem(tc_pipe_kernel<KS, MODE>, G::kSmem, opt_in);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(plan.grid); cfg.blockDim = dim3(G::kThreads); cfg.dynamicSmemBytes = G::kSmem; cfg.stream = st;
    // the pipelines of different CTAs wait on one another's results: all CTAs have to be resident at once
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc_pipe_kernel<KS, MODE>, tmK, tmVs, tmQ, tmVh, prm);
}

}  // namespace

// Work split of the one-kernel forward: CTAs, state tiles per plane, token splits per plane, and whether the
// planes are applied in order with the state pipeline running a bounded number of planes ahead.
PipePlan plan_pipe(int BH, int rows, int cols, int gridH) {
    PipePlan pl;
    const int sms = device_sm_count();
    if (rows < 1) rows = 1;  // size queries reach here with shapes the kernel never takes
    if (BH < 1) BH = 1;
    pl.s_tiles = (rows + kSTile - 1) / kSTile;
    const int patches = ((cols + kTX - 1) / kTX) * ((gridH + kTY - 1) / kTY);
    // splits: about eight tiles each, but at least enough to give every CTA a share when there are few planes
    int P = pl.s_tiles / 8;
    const int spread = sms / BH;
    if (P < spread) P = spread;
    if (P > pl.s_tiles) P = pl.s_tiles;
    if (P > kPipeMaxSplits) P = kPipeMaxSplits;
    if (P < 1) P = 1;
    pl.s_per = (pl.s_tiles + P - 1) / P;
    pl.P = (pl.s_tiles + pl.s_per - 1) / pl.s_per;
    const long long items = (long long)BH * pl.P, total_patches = (long long)BH * patches;
    long long want = items > total_patches ? items : total_patches;
    pl.grid = (int)(want < sms ? want : sms);
    // V of all planes beyond what L2 can hold until it is applied: walk the planes in order
    const long long v_bytes = (long long)BH * rows * 128;
    const long long budget = 40ll << 20;
    pl.plane_order = (v_bytes > budget && patches >= pl.grid) ? 1 : 0;
    long long ahead = budget / ((long long)rows * 128);
    if (ahead < 1) ahead = 1;
    pl.ahead = pl.plane_order ? (int)(ahead < BH ? ahead : BH) : BH;
    return pl;
}

cudaError_t launch_pipe(const Problem& p, float* partial, float* state, unsigned* ctr, unsigned* status, cudaStream_t st) {
    if (p.d == 32)
        return p.ksize == 3 ? launch_pipe_ks<3, 1>(p, partial, state, ctr, status, st)
                            : launch_pipe_ks<5, 1>(p, partial, state, ctr, status, st);
    if (p.blockdiag)
        return p.ksize == 3 ? launch_pipe_ks<3, 2>(p, partial, state, ctr, status, st)
                            : launch_pipe_ks<5, 2>(p, partial, state, ctr, status, st);
    return p.ksize == 3 ? launch_pipe_ks<3, 0>(p, partial, state, ctr, status, st)
                        : launch_pipe_ks<5, 0>(p, partial, state, ctr, status, st);
}

}  // namespace tc
}  // namespace castling

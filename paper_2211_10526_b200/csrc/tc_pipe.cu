// Whole forward pass of the tensor-core path as ONE persistent kernel (bf16; width-64 heads, or width-32
// heads packed two to a 128-byte row), an alternative to the separate state and apply kernels:
//     S = sum_n k^_n^T v_n,  s = sum_n v_n            (state, per (b,h))
//     out_t = (1/pi) q^_t S + 1/2 s + bias + DWConv(V)_t                              (Eq. 9)
// One CTA per multiprocessor, launched cooperatively so that all CTAs are resident.  Every CTA runs two
// pipelines side by side, in different warps, and takes its work from two counters in global memory, in plane
// order (a plane is one (b,h)): chunks of rows for the state pipeline, patches of the token grid for the
// apply pipeline.  A slower multiprocessor simply takes fewer.
//   state pipeline   warp 2 (claims chunks; TMA: K and V tiles of 64 rows), warp 3 lane 0 (UMMAs, A = [K^ ; 1 0 0 ...]
//                    so that accumulator row 64 is the token sum of V), warps 12..15 (scale every K row by
//                    1 / max(||k||, eps) in place; add the chunk's sums to the plane's state in memory with
//                    vector atomics), warp 3 lane 1 (counts the chunk once its sums are on their way)
//   apply pipeline   warp 0 (claims patches; TMA: Q patch and V patch with halo; per plane S' and 1/2 s), warp 1
//                    (UMMAs: acc = Q S'), conv warps (depthwise convolution of the V patch on CUDA cores, lane =
//                    channel pair; result plus 1/2 s and the bias staged in shared memory as fp32), warps 4..11
//                    (||q||, accumulator row scaled by 1/||q|| plus the staged row, one rounding to bf16, patch
//                    stored with TMA)
// The CTA that counts the last chunk of a plane finishes it: its norm warps turn the sums into the bf16
// operand image S' = S / pi and 1/2 s, write both to memory and raise the plane's flag; the apply producers of
// all CTAs wait for that flag when they first take a patch of the plane and copy the block into shared memory.
// The states are cleared by the kernel itself.  The sums of a plane are added in the order the chunks happen
// to finish, so the result varies in the last bits from run to run (the separate kernels add in a fixed order).
// The state pipeline keeps a bounded number of planes ahead of the apply pipeline, so that the V rows the
// apply pipeline needs were read moments ago and are served from L2: V comes from HBM once.
// Flags are polled by one thread per CTA (many pollers on one address queue up at its L2 slice and slow every
// other access to that slice); the other threads sleep on a shared-memory barrier that thread completes.
// Every wait is bounded; a wait that runs out raises a bit in the status word, and every CTA that sees the
// bit leaves.
#include "tc_common.cuh"
#include "tc_host.cuh"

namespace castling {
namespace tc {
namespace {

constexpr int kD = 64;
constexpr int kTY = 8, kTX = 16;            // patch: 8 rows x 16 columns of 128-byte rows
constexpr int kPatch = kTY * kTX;
constexpr int kQBytes = kPatch * kD * 2;    // 16 KiB
constexpr int kStgStride = kD * 4;          // fp32 row; 16-byte chunk c of row t sits at chunk c ^ (t & 7)
constexpr int kStgBytes = kPatch * kStgStride;
constexpr int kSpBytes = kD * kD * 2;       // S' = S / pi as the bf16 B operand of the apply UMMAs (swizzled image)
constexpr int kHsBytes = kD * 4;            // 1/2 s
constexpr int kReadyWords = (kSpBytes + kHsBytes) / 4;  // per plane in global memory: S' image, then 1/2 s
constexpr int kEpiWarps = 8, kEpiThreads = kEpiWarps * 32;
constexpr int kNormWarps = 4, kNormThreads = kNormWarps * 32;
constexpr int kSTile = 64;                  // rows per state stage
constexpr int kSTileBytes = kSTile * 128;   // 8 KiB per operand tile
constexpr int kSStage = 2 * kSTileBytes;    // K then V
constexpr int kOnesBytes = 2048;
constexpr int kTmemCols = 256;              // [0,128): two apply accumulators; [128,256): two state accumulators
constexpr int kWords = kD * kD + kD;        // one state: S then s
constexpr int kWords4 = kWords / 4;
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
    static constexpr int kStages = 2;                      // apply stages (Q patch + V patch with halo)
    static constexpr int kSStages = (KS == 3) ? 3 : 2;     // state stages (K tile + V tile)
    // S' x2 | out patch | apply stages | staging x2 | state stages | ones | rq x2 | 1/2 s x2 | barriers
    static constexpr int kOffS = 0, kOffOut = 2 * kSpBytes, kOffStages = kOffOut + kQBytes;
    static constexpr int kOffStg = kOffStages + kStages * kStage;
    static constexpr int kOffSStages = ((kOffStg + 2 * kStgBytes + 1023) / 1024) * 1024;
    static constexpr int kOffOnes = kOffSStages + kSStages * kSStage;
    static constexpr int kOffRq = kOffOnes + kOnesBytes;   // sum of squares of each half of a Q row
    static constexpr int kOffHs = kOffRq + 2 * kPatch * 4;
    static constexpr int kOffBar = kOffHs + 2 * kHsBytes;
    static constexpr size_t kSmem = kOffBar + 512;
    static_assert(kSmem <= 227 * 1024, "shared memory of the one-kernel forward");
};

struct PipeParams {
    float* state;                  // [BH][kWords] sums S then s of every plane
    float* ready;                  // [BH][kReadyWords] what the apply pipelines load per plane: S' image, 1/2 s
    unsigned* ctr;                 // kPipeCtrHeader words, then kPipeCtrPerPlane per plane; all zero between calls
    const __nv_bfloat16* w;        // [H*d][KS][KS]
    const __nv_bfloat16* bias;     // [H*d] or nullptr
    int flat;                      // the planes have one uniform stride: the apply tensor maps are 4-D
    int H, head0, BH, hdiv;
    int tilesX, tilesY;            // patches per plane
    int s_tiles;                   // 64-row state tiles per plane
    int chunk_tiles, n_chunks;     // tiles per chunk, chunks per plane
    int ahead;                     // a chunk of plane p is started only when plane p - ahead is applied
    float eps2;
    unsigned* status;
};

constexpr int kNoWork = -1;            // stage info: nothing more to do

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Adds one to a counter in global memory, ordered after every write that happens before the call: the caller's own
// and, through a preceding CTA barrier, those of the other threads of the CTA.  One releasing thread per CTA: a
// device-wide fence in every thread waits for the copies the CTA's pipelines have in flight, again and again.
__device__ __forceinline__ void signal_add(unsigned* p) {
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}

// Adds four floats to four consecutive words of global memory (performed at the L2, no value returned).
__device__ __forceinline__ void red_add_f32x4(float* p, float a, float b, float c, float d) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// The same with the old value returned, and ordered before what follows as well.
__device__ __forceinline__ unsigned signal_add_fetch(unsigned* p) {
    unsigned old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(p) : "memory");
    return old;
}

// Copy `bytes` (a multiple of 16) from global to shared memory; completion is counted on `bar`.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Bounded wait for a counter in global memory to reach `want`.  Gives up (returns false) when the limit
// runs out (raising the status bit), when this CTA has given up elsewhere, or when any CTA has raised a bit.
__device__ __forceinline__ bool wait_counter(const unsigned* p, unsigned want, volatile int* abort_flag, unsigned* status) {
    if (ld_acquire(p) >= want) return true;
    const unsigned long long t0 = global_ns();
    uint32_t spins = 0;
    while (true) {
        __nanosleep(200);
        if (ld_acquire(p) >= want) return true;
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

// MODE 0: width-64 heads; 1: width-32 heads, two adjacent tokens per 128-byte row; 2: two width-32 heads side
// by side in one row (block-diagonal state).
template <int KS, int MODE>
__global__ void __launch_bounds__((PGeo<KS, MODE == 1>::kThreads), 1)
tc_pipe_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmVs,
               const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmVh,
               const __grid_constant__ CUtensorMap tmO, const PipeParams prm) {
    constexpr bool PAIR = (MODE == 1), BLOCKDIAG = (MODE == 2), HALVES = PAIR || BLOCKDIAG;
    using G = PGeo<KS, PAIR>;
    constexpr int NA = G::kStages, NS = G::kSStages;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* S_s = smem + G::kOffS;
    uint8_t* out_s = smem + G::kOffOut;
    uint8_t* stg = smem + G::kOffStg;
    uint8_t* stages = smem + G::kOffStages;
    uint8_t* sstages = smem + G::kOffSStages;
    uint8_t* ones = smem + G::kOffOnes;
    float* rq_s = reinterpret_cast<float*>(smem + G::kOffRq);
    float* hs_s = reinterpret_cast<float*>(smem + G::kOffHs);   // [2][64] 1/2 s of the plane in S' buffer 0 / 1
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + G::kOffBar);
    uint64_t* a_full = bars;                 // [NA] Q and V patch landed
    uint64_t* a_empty = a_full + NA;         // [NA] stage consumed (conv + epilogue warps, UMMA commit)
    uint64_t* acc_full = a_empty + NA;       // [2]  apply UMMAs retired
    uint64_t* conv_full = acc_full + 2;      // [2]  staging written (conv threads)
    uint64_t* buf_free = conv_full + 2;      // [2]  accumulator and staging read out (epilogue threads)
    uint64_t* sp_full = buf_free + 2;        // [2]  S' and 1/2 s of a plane landed
    uint64_t* sig_bar = sp_full + 2;         //      a chunk's sums are on their way to the plane's state (norm threads)
    uint64_t* s_full = sig_bar + 1;          // [NS] K and V tile landed
    uint64_t* s_scaled = s_full + NS;        // [NS] K rows normalised
    uint64_t* s_empty = s_scaled + NS;       // [NS] state UMMAs of the stage retired
    uint64_t* sacc_full = s_empty + NS;      // [2]  accumulation of a plane retired
    uint64_t* sacc_free = sacc_full + 2;     // [2]  accumulator read out
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sacc_free + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* last_slot = reinterpret_cast<int*>(tmem_slot + 2);
    unsigned* applied_s = reinterpret_cast<unsigned*>(tmem_slot + 4);  // [8] conv warps done with the CTA's i-th patch, slot i & 7
    volatile int* a_info = reinterpret_cast<volatile int*>(tmem_slot + 12);  // [NA] patch in the apply stage, or kNoWork
    volatile int* s_info = a_info + 4;                                      // [NS] chunk * 4 + (first tile) + 2 * (last tile), or kNoWork
    volatile int* sig_info = s_info + 4;     // [4] plane of the k-th chunk this CTA has summed (slot k & 3), or kNoWork
    volatile int* fin_req = sig_info + 4;    // [4] planes whose sums are complete and that this CTA is to finish (slot i & 3)
    volatile int* fin_head = fin_req + 4;    // [2] number of such requests so far; 1 when the signalling thread has left
    volatile int* sig_tail = fin_head + 6;   // [2] chunk counts the signalling thread has taken over; planes finished by the norm warps

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_cta = (int)gridDim.x, cta = (int)blockIdx.x;
    unsigned* plane_ctr = prm.ctr + kPipeCtrHeader;
    const int tpb = prm.tilesX * prm.tilesY;                 // patches per plane
    const int n_patches = prm.BH * tpb, n_chunks_all = prm.BH * prm.n_chunks;

    if (tid == 0) {
        for (int s = 0; s < NA; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], G::kConvThreads + kEpiThreads + 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1); mbar_init(&conv_full[b], G::kConvThreads); mbar_init(&buf_free[b], kEpiThreads);
            mbar_init(&sacc_full[b], 1); mbar_init(&sacc_free[b], kNormThreads);
        }
        mbar_init(&sp_full[0], 1); mbar_init(&sp_full[1], 1); mbar_init(sig_bar, kNormThreads);
        fin_head[0] = 0; fin_head[1] = 0; sig_tail[0] = 0; sig_tail[1] = 0;
        for (int s = 0; s < NS; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_scaled[s], kNormThreads); mbar_init(&s_empty[s], 1); }
        *abort_flag = 0;
        for (int i = 0; i < 8; ++i) applied_s[i] = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmVs); tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmVh); tma_prefetch_desc(&tmO);
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
    // Every CTA clears its part of the states, which the chunk sums are added to; the first addition of any CTA
    // waits until all parts are cleared (by then they long are).
    {
        const int n4 = prm.BH * kWords4;
        float4* st4 = reinterpret_cast<float4*>(prm.state);
        for (int i = (int)((long long)n4 * cta / n_cta) + tid, e = (int)((long long)n4 * (cta + 1) / n_cta); i < e; i += blockDim.x)
            st4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    if (tid == 0) signal_add(prm.ctr + kPipeCtrCleared);
    const uint32_t tmem = *tmem_slot;
    const uint32_t tmem_state = tmem + 128;

    if (warp == 0) {
        // ================= apply pipeline: TMA producer =================
        if (lane == 0) {
            int issued = 0;
            const uint64_t pol_q = l2_policy_evict_first();  // Q is read once
            // Patches are handed out one at a time, in plane order, from a counter in global memory: a slower
            // multiprocessor simply takes fewer.  The next claim is under way while this patch is loaded.
            int g = (int)atomicAdd(prm.ctr + kPipeCtrNextPatch, 1u);
            int prev_bh = -1, seg = 0;
            for (int it = 0;; ++it) {
                const int s = it % NA, use = it / NA;
                if (use > 0 && !mbar_wait(&a_empty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) break;
                if (g >= n_patches) {  // tell the other roles that this was all
                    a_info[s] = kNoWork;
                    mbar_arrive(&a_full[s]);
                    break;
                }
                const int g_next = (int)atomicAdd(prm.ctr + kPipeCtrNextPatch, 1u);
                if (g_next < n_patches) {
                    // the next patch's Q on its way from memory to L2 already: the stages hold too little to cover
                    // that latency (V was read by the state pipeline moments ago and is in L2 anyway)
                    const int nb = g_next / tpb, nr = g_next - nb * tpb;
                    const int ny = (nr / prm.tilesX) * kTY, nx = (nr % prm.tilesX) * kTX;
                    if (prm.flat) tma_prefetch_4d(&tmQ, 0, nx, ny, nb);
                    else tma_prefetch_5d(&tmQ, 0, nx, ny, nb % prm.hdiv, nb / prm.hdiv);
                }
                const int bh = g / tpb, rem = g - bh * tpb;
                if (bh != prev_bh) {
                    // a new plane: its S' and 1/2 s, once they are ready, into the S' buffer that the plane before
                    // the previous one used (every patch of that plane has left its stage: see the wait above)
                    prev_bh = bh;
                    if (!wait_counter(plane_ctr + (size_t)bh * kPipeCtrPerPlane + kPipeCtrReady, 1u, abort_flag, prm.status)) break;
                    asm volatile("fence.proxy.async;" ::: "memory");
                    const float* blk = prm.ready + (size_t)bh * kReadyWords;
                    mbar_expect_tx(&sp_full[seg & 1], kSpBytes + kHsBytes);
                    bulk_load(S_s + (seg & 1) * kSpBytes, blk, kSpBytes, &sp_full[seg & 1]);
                    bulk_load(hs_s + (seg & 1) * kD, blk + kSpBytes / 4, kHsBytes, &sp_full[seg & 1]);
                    ++seg;
                }
                const int y0 = (rem / prm.tilesX) * kTY, x0 = (rem % prm.tilesX) * kTX;
                uint8_t* qs = stages + s * G::kStage;
                a_info[s] = g;
                mbar_expect_tx(&a_full[s], kQBytes + G::kVBytes);
                if (prm.flat) {
                    tma_load_4d_hint(qs, &tmQ, &a_full[s], 0, x0, y0, bh, pol_q);
                    tma_load_4d(qs + kQBytes, &tmVh, &a_full[s], 0, x0 - G::HC, y0 - G::R, bh);
                } else {
                    const int pb = bh / prm.hdiv, ph = bh - pb * prm.hdiv;
                    tma_load_5d_hint(qs, &tmQ, &a_full[s], 0, x0, y0, ph, pb, pol_q);
                    tma_load_5d(qs + kQBytes, &tmVh, &a_full[s], 0, x0 - G::HC, y0 - G::R, ph, pb);
                }
                ++issued;
                g = g_next;
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
            uint32_t s_addr = smem_u32(S_s);
            int prev_bh = -1, seg = 0;
            for (int it = 0;; ++it) {
                const int s = it % NA, use = it / NA, b = it & 1, ub = it >> 1;
                if (!mbar_wait(&a_full[s], use & 1, abort_flag, prm.status, kBit)) break;
                const int g = a_info[s];
                if (g == kNoWork) break;
                const int bh = g / tpb;
                if (bh != prev_bh) {
                    if (!mbar_wait(&sp_full[seg & 1], (seg >> 1) & 1, abort_flag, prm.status, kBit)) break;
                    s_addr = smem_u32(S_s) + (seg & 1) * kSpBytes;
                    ++seg; prev_bh = bh;
                }
                if (ub > 0 && !mbar_wait(&buf_free[b], (ub - 1) & 1, abort_flag, prm.status, kBit)) break;
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
            bool ok = true;
            // Chunks of rows are handed out like the patches, in plane order.
            int g = (int)atomicAdd(prm.ctr + kPipeCtrNextChunk, 1u);
            while (ok) {
                if (g >= n_chunks_all) {
                    const int s = issued % NS, use = issued / NS;
                    if (use > 0 && !mbar_wait(&s_empty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) break;
                    s_info[s] = kNoWork;
                    mbar_arrive(&s_full[s]);
                    break;
                }
                const int g_next = (int)atomicAdd(prm.ctr + kPipeCtrNextChunk, 1u);
                if (g_next < n_chunks_all) {
                    // the next chunk's rows on their way from memory to L2 already (see the patches above)
                    const int np = g_next / prm.n_chunks, nj = g_next - np * prm.n_chunks;
                    const int nb = np / prm.hdiv, nh = np - nb * prm.hdiv;
                    const int n0 = nj * prm.chunk_tiles, n1 = min(prm.s_tiles, n0 + prm.chunk_tiles);
                    for (int t = n0; t < n1; ++t) {
                        tma_prefetch_4d(&tmK, 0, t * kSTile, nh, nb);
                        tma_prefetch_4d(&tmVs, 0, t * kSTile, nh, nb);
                    }
                }
                const int plane = g / prm.n_chunks, j = g - plane * prm.n_chunks;
                if (plane >= prm.ahead &&
                    !wait_counter(plane_ctr + (size_t)(plane - prm.ahead) * kPipeCtrPerPlane + kPipeCtrApplied, (unsigned)tpb,
                                  abort_flag, prm.status)) break;
                const int pb = plane / prm.hdiv, ph = plane - pb * prm.hdiv;
                const int t0 = j * prm.chunk_tiles, t1 = min(prm.s_tiles, t0 + prm.chunk_tiles);
                for (int t = t0; t < t1; ++t, ++issued) {
                    const int s = issued % NS, use = issued / NS;
                    if (use > 0 && !mbar_wait(&s_empty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) { ok = false; break; }
                    uint8_t* ks = sstages + s * kSStage;
                    s_info[s] = g * 4 + (t == t0 ? 1 : 0) + (t == t1 - 1 ? 2 : 0);
                    mbar_expect_tx(&s_full[s], kSStage);
                    tma_load_4d_hint(ks, &tmK, &s_full[s], 0, t * kSTile, ph, pb, pol_k);
                    tma_load_4d_hint(ks + kSTileBytes, &tmVs, &s_full[s], 0, t * kSTile, ph, pb, pol_v);
                }
                g = g_next;
            }
            if (*abort_flag) {
                for (int i = max(0, issued - NS); i < issued; ++i)
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&s_full[i % NS], (i / NS) & 1); ++spin) {}
            }
        }
    } else if (warp == 3) {
        if (lane == 1) {
            // ================= state pipeline: signalling thread =================
            // Counts every chunk of this CTA once its sums are on their way (ordered after them), so that the
            // threads that produced them need not wait for memory to acknowledge anything.  Whoever counts the
            // last chunk of a plane has its CTA finish that plane (see the norm warps).
            for (int k = 0;; ++k) {
                if (!mbar_wait(sig_bar, k & 1, abort_flag, prm.status, kBit)) break;
                const int plane = sig_info[k & 3];
                __threadfence_block();
                sig_tail[0] = k + 1;  // the norm warps complete the barrier's next phase only after this
                if (plane == kNoWork) break;
                const unsigned old = signal_add_fetch(plane_ctr + (size_t)plane * kPipeCtrPerPlane + kPipeCtrWritten);
                if (old == (unsigned)prm.n_chunks - 1u) {
                    const int h = fin_head[0];
                    for (uint32_t spin = 0; h - sig_tail[1] >= 4 && spin < (1u << 22) && !*abort_flag; ++spin) __nanosleep(100);
                    fin_req[h & 3] = plane;
                    __threadfence_block();
                    fin_head[0] = h + 1;
                }
            }
            __threadfence_block();
            fin_head[1] = 1;
        } else if (lane == 0) {
            // ================= state pipeline: UMMA issuer =================
            constexpr uint32_t idesc = umma_idesc_bf16(128, kD, true, true);
            const uint32_t ones_addr = smem_u32(ones);
            int k_chunk = 0;  // chunks started so far
            for (int gt = 0;; ++gt) {
                const int s = gt % NS, use = gt / NS;
                if (!mbar_wait(&s_scaled[s], use & 1, abort_flag, prm.status, kBit)) break;
                const int info = s_info[s];
                if (info == kNoWork) break;
                const bool first = (info & 1) != 0, last = (info & 2) != 0;
                if (first) ++k_chunk;
                const int buf = (k_chunk - 1) & 1;
                if (first && k_chunk > 2 && !mbar_wait(&sacc_free[buf], (((k_chunk - 1) >> 1) - 1) & 1, abort_flag, prm.status, kBit)) break;
                tcgen05_fence_after_sync();
                const uint32_t ka = smem_u32(sstages + s * kSStage), va = ka + kSTileBytes;
#pragma unroll
                for (int j = 0; j < kSTile / 16; ++j) {  // one UMMA per 16 rows (K = 16)
                    const uint32_t a0 = ka + j * 2048, b0 = va + j * 2048;
                    umma_bf16(tmem_state + buf * kD, umma_desc_sw128(a0, ones_addr - a0, 1024),
                              umma_desc_sw128(b0, 0, 1024), idesc, !first || (j != 0));
                }
                umma_commit(&s_empty[s]);
                if (last) umma_commit(&sacc_full[buf]);
            }
        }
    } else if (warp < kFirstWarpNorm) {
        // ================= apply pipeline: epilogue, thread = (token row of the patch, half of the channels) =================
        const int quarter = warp & 3, row = quarter * 32 + lane, et = tid - 32 * kFirstWarpEpi;
        const int half = (warp - kFirstWarpEpi) >> 2;  // channels half*32 .. half*32 + 31
        const bool leader = (et == 0);
        const uint64_t pol_o = l2_policy_evict_first();  // the output is not read back here
        bool failed = false;  // the same for every epilogue thread wherever a barrier follows
        for (int it = 0;; ++it) {
            const int b = it & 1, ub = it >> 1, s = it % NA, use = it / NA;
            // every epilogue thread learns the stage's patch (or that there is none, or that a wait failed)
            if (barrier_any(1, kEpiThreads, !mbar_wait(&a_full[s], use & 1, abort_flag, prm.status, kBit))) break;
            const int g = a_info[s];
            if (g == kNoWork) break;
            const int bh = g / tpb, rem = g - bh * tpb;
            float a[32];
            if (!failed) {
                // this thread's half of sum(q^2) for its token; the other half comes from the partner warp
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
                rq_s[half * kPatch + row] = (ss[0] + ss[1]) + (ss[2] + ss[3]);
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
                failed = __any_sync(0xffffffffu, !mbar_wait(&conv_full[b], ub & 1, abort_flag, prm.status, kBit));
            }
            // the previous patch's TMA store must have read out_s before it is rewritten; the same barrier makes
            // both halves of every row's sum of squares visible and tells every thread whether one has given up
            if (it > 0 && leader) tma_store_wait_read();
            if (barrier_any(1, kEpiThreads, failed)) break;
            const float rq = HALVES ? rsqrtf(fmaxf(rq_s[half * kPatch + row], prm.eps2))   // half row = one token / one head
                                    : rsqrtf(fmaxf(rq_s[row] + rq_s[kPatch + row], prm.eps2));
            const uint8_t* srow = stg + b * kStgBytes + row * kStgStride;
            uint8_t* orow = out_s + row * 128;
#pragma unroll
            for (int e = 0; e < 4; ++e) {  // 8 channels -> one 16-byte chunk of the bf16 row
                const float4 c0 = *reinterpret_cast<const float4*>(srow + (((half * 8 + 2 * e) ^ (row & 7)) << 4));
                const float4 c1 = *reinterpret_cast<const float4*>(srow + (((half * 8 + 2 * e + 1) ^ (row & 7)) << 4));
                uint4 pk;
                pk.x = pack_bf16x2(fmaf(a[8 * e + 0], rq, c0.x), fmaf(a[8 * e + 1], rq, c0.y));
                pk.y = pack_bf16x2(fmaf(a[8 * e + 2], rq, c0.z), fmaf(a[8 * e + 3], rq, c0.w));
                pk.z = pack_bf16x2(fmaf(a[8 * e + 4], rq, c1.x), fmaf(a[8 * e + 5], rq, c1.y));
                pk.w = pack_bf16x2(fmaf(a[8 * e + 6], rq, c1.z), fmaf(a[8 * e + 7], rq, c1.w));
                *reinterpret_cast<uint4*>(orow + (((half * 4 + e) ^ (row & 7)) << 4)) = pk;
            }
            tcgen05_fence_before_sync();
            mbar_arrive(&buf_free[b]);
            fence_proxy_async_smem();
            named_barrier_sync(1, kEpiThreads);
            if (leader) {
                const int y0 = (rem / prm.tilesX) * kTY, x0 = (rem % prm.tilesX) * kTX;
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
    } else if (warp < kFirstWarpConv) {
        // ================= state pipeline: K normalisation, accumulator read-out =================
        const int t = tid - 32 * kFirstWarpNorm;   // 0..127: row t >> 1 of the stage, half t & 1 of that row
        const int quarter = warp & 3;
        const int r = t >> 1, hf = t & 1;
        volatile int* fin_seen = fin_head + 2;  // [4] what thread 0 saw of fin_head, for everybody
        int k_chunk = 0;   // chunks started so far
        int fin_done = 0;  // planes finished by this CTA so far
        bool dead = false; // a wait has failed: the same for all norm threads wherever a barrier follows
        // Finishes a plane whose sums are complete: S' = S / pi as the bf16 operand image of the apply UMMAs (16-byte
        // chunk c of row i at chunk c ^ (i & 7)) and 1/2 s go to memory, where the apply pipelines of all CTAs copy
        // them from; then the plane's flag is raised.
        auto finish_plane = [&](int plane) {
            const float* st = prm.state + (size_t)plane * kWords;
            uint8_t* blk = reinterpret_cast<uint8_t*>(prm.ready + (size_t)plane * kReadyWords);
            const int i = t >> 1;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const int c = (t & 1) * 4 + cc, col = c * 8;
                float4 lo, hi;
                if (!PAIR) {
                    const float4* src = reinterpret_cast<const float4*>(st + i * kD + col);
                    lo = __ldcg(src); hi = __ldcg(src + 1);
                    if (BLOCKDIAG && ((i < 32) != (col < 32))) {  // off-diagonal block: the other head's keys
                        lo = make_float4(0.f, 0.f, 0.f, 0.f); hi = lo;
                    }
                } else if ((i < 32) == (col < 32)) {
                    // operand = blockdiag(S32, S32) with S32 = block(0,0) + block(1,1) of the paired sums
                    const int a = i & 31, bcol = col & 31;
                    const float4* s0 = reinterpret_cast<const float4*>(st + a * kD + bcol);
                    const float4* s1 = reinterpret_cast<const float4*>(st + (32 + a) * kD + 32 + bcol);
                    const float4 l0 = __ldcg(s0), h0 = __ldcg(s0 + 1), l1 = __ldcg(s1), h1 = __ldcg(s1 + 1);
                    lo = make_float4(l0.x + l1.x, l0.y + l1.y, l0.z + l1.z, l0.w + l1.w);
                    hi = make_float4(h0.x + h1.x, h0.y + h1.y, h0.z + h1.z, h0.w + h1.w);
                } else {
                    lo = make_float4(0.f, 0.f, 0.f, 0.f); hi = lo;
                }
                uint4 o;
                o.x = pack_bf16x2(lo.x * kInvPi, lo.y * kInvPi); o.y = pack_bf16x2(lo.z * kInvPi, lo.w * kInvPi);
                o.z = pack_bf16x2(hi.x * kInvPi, hi.y * kInvPi); o.w = pack_bf16x2(hi.z * kInvPi, hi.w * kInvPi);
                *reinterpret_cast<uint4*>(blk + i * 128 + ((c ^ (i & 7)) << 4)) = o;
            }
            if (t < kD) {
                const float* sv = st + kD * kD;
                const float h = PAIR ? 0.5f * (__ldcg(sv + (t & 31)) + __ldcg(sv + 32 + (t & 31))) : 0.5f * __ldcg(sv + t);
                reinterpret_cast<float*>(blk + kSpBytes)[t] = h;
            }
            named_barrier_sync(2, kNormThreads);
            if (t == 0) { signal_add(plane_ctr + (size_t)plane * kPipeCtrPerPlane + kPipeCtrReady); sig_tail[1] = sig_tail[1] + 1; }
        };
        for (int gt = 0;; ++gt) {
            const int s = gt % NS, use = gt / NS;
            if (t == 0) fin_seen[gt & 1] = fin_head[0];
            // every thread learns the stage's chunk (or that there is none, or that a wait failed)
            if (barrier_any(3, kNormThreads, dead || !mbar_wait(&s_full[s], use & 1, abort_flag, prm.status, kBit))) { dead = true; break; }
            while (fin_done < fin_seen[gt & 1]) { finish_plane(fin_req[fin_done & 3]); ++fin_done; }
            const int info = s_info[s];
            if (info == kNoWork) { mbar_arrive(&s_scaled[s]); break; }  // passes the word on to the UMMA issuer
            const bool first = (info & 1) != 0, last = (info & 2) != 0;
            if (first) ++k_chunk;
            {
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
            if (!last) continue;
            // the chunk's sums leave TMEM (rows 0..63 are S, row 64 is s) and are added to the plane's state
            const int chunk = info >> 2, plane = chunk / prm.n_chunks;
            const int buf = (k_chunk - 1) & 1;
            bool ok = mbar_wait(&sacc_full[buf], ((k_chunk - 1) >> 1) & 1, abort_flag, prm.status, kBit);
            // the first sums of this CTA: every CTA must have cleared its part of the states by now
            if (k_chunk == 1 && t == 0 && ok) ok = wait_counter(prm.ctr + kPipeCtrCleared, (unsigned)n_cta, abort_flag, prm.status);
            if (barrier_any(2, kNormThreads, !ok)) { dead = true; continue; }  // everybody, or nobody
            tcgen05_fence_after_sync();
            float* dst = prm.state + (size_t)plane * kWords;
            if (quarter < 3) {
                const int row = quarter * 32 + lane;
#pragma unroll
                for (int cc = 0; cc < kD / 16; ++cc) {
                    float v[16];
                    tmem_ld16(tmem_state + ((uint32_t)(quarter * 32) << 16) + buf * kD + cc * 16, v);
                    tmem_ld_wait();
                    if (row <= kD) {
                        float* o4 = dst + row * kD + cc * 16;  // row 64 lands on s
#pragma unroll
                        for (int e = 0; e < 4; ++e) red_add_f32x4(o4 + 4 * e, v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                    }
                }
            }
            tcgen05_fence_before_sync();
            mbar_arrive(&sacc_free[buf]);
            // the signalling thread counts the chunk, ordered after these additions; it has to have seen the previous
            // phase of its barrier complete before this one may (a waiter can be one phase behind, not two)
            if (t == 0) {
                for (uint32_t spin = 0; sig_tail[0] < k_chunk - 1 && spin < (1u << 22) && !*abort_flag; ++spin) __nanosleep(100);
                sig_info[(k_chunk - 1) & 3] = plane;
            }
            named_barrier_sync(2, kNormThreads);
            mbar_arrive(sig_bar);
        }
        if (!dead) {
            // no more chunks: the signalling thread leaves after the last count; planes may still come up for finishing
            if (t == 0) {
                for (uint32_t spin = 0; sig_tail[0] < k_chunk && spin < (1u << 22) && !*abort_flag; ++spin) __nanosleep(100);
                sig_info[k_chunk & 3] = kNoWork;
            }
            named_barrier_sync(2, kNormThreads);
            mbar_arrive(sig_bar);
            const unsigned long long t_start = global_ns();
            while (true) {
                if (t == 0) {
                    const int left = fin_head[1];
                    __threadfence_block();
                    fin_seen[2] = fin_head[0]; fin_seen[3] = left;
                    if (!left && (*abort_flag || global_ns() - t_start > kWaitLimitNs)) { fin_seen[3] = 2; *abort_flag = 1; atomicOr(prm.status, kBit); }
                }
                named_barrier_sync(2, kNormThreads);
                const int seen = fin_seen[2], left = fin_seen[3];
                named_barrier_sync(2, kNormThreads);
                if (left != 2) while (fin_done < seen) { finish_plane(fin_req[fin_done & 3]); ++fin_done; }
                if (left) break;
                __nanosleep(200);
            }
        }
    } else {
        // ================= apply pipeline: depthwise convolution =================
        const int cwi = warp - kFirstWarpConv;
        const int cw = cwi >> 1, xh = cwi & 1;  // row group and column half of the patch
        constexpr int kCX = kTX / 2;
        constexpr int R = G::R, RO = G::kConvRows, ROWS = RO + 2 * R;
        float2 wreg[KS][KS];
        float2 cinit = make_float2(0.f, 0.f);
        int prev_bh = -1, pseg = 0;
        for (int it = 0;; ++it) {
            const int s = it % NA, use = it / NA, b = it & 1, ub = it >> 1;
            if (__any_sync(0xffffffffu, !mbar_wait(&a_full[s], use & 1, abort_flag, prm.status, kBit))) break;
            const int g = a_info[s];
            if (g == kNoWork) break;
            const int bh = g / tpb;
            if (bh != prev_bh) {
                prev_bh = bh;
                // the plane's 1/2 s arrives with its S'
                if (__any_sync(0xffffffffu, !mbar_wait(&sp_full[pseg & 1], (pseg >> 1) & 1, abort_flag, prm.status, kBit))) break;
                const float* hs = hs_s + (pseg & 1) * kD;
                ++pseg;
                // this lane's channel pair: 2*lane of 64 channels, or (PAIR) 2*(lane & 15) of 32 channels
                // for the token of parity lane >> 4
                const int cp2 = PAIR ? 2 * (lane & 15) : 2 * lane;
                const int ch = ((prm.head0 + bh) % prm.H) * (PAIR ? 32 : kD) + cp2;
                cinit.x = hs[cp2]; cinit.y = hs[cp2 + 1];
                if (prm.bias) { cinit.x += __bfloat162float(prm.bias[ch]); cinit.y += __bfloat162float(prm.bias[ch + 1]); }
#pragma unroll
                for (int dy = 0; dy < KS; ++dy)
#pragma unroll
                    for (int dx = 0; dx < KS; ++dx)
                        wreg[dy][dx] = make_float2(__bfloat162float(prm.w[(size_t)ch * KS * KS + dy * KS + dx]),
                                                   __bfloat162float(prm.w[(size_t)(ch + 1) * KS * KS + dy * KS + dx]));
            }
            if (ub > 0 && __any_sync(0xffffffffu, !mbar_wait(&buf_free[b], (ub - 1) & 1, abort_flag, prm.status, kBit))) break;
            // Window of KS tokens per halo row, sliding along x.  Token t (relative to the first token this
            // lane needs) sits U bytes after token t-1: U = 128, one token per column, or (PAIR) 64.
            // One output column advances the window by STEP tokens (2 when PAIR: the lane's token keeps
            // its parity).  Slot of token t in the rotating window: t % KS (t is a compile-time value).
            constexpr int U = PAIR ? 64 : 128, STEP = PAIR ? 2 : 1;
            const int tok0 = PAIR ? 2 * (xh * kCX + G::HC) + (lane >> 4) - R : xh * kCX;
            const uint8_t* vh = stages + s * G::kStage + kQBytes + (RO * cw) * G::HX * 128 + tok0 * U +
                                (PAIR ? (lane & 15) * 4 : lane * 4);
            // fp32 rows of the staging buffer: 16-byte chunk c of patch token t at chunk c ^ (t & 7); t & 7 = x below
            uint8_t* so = stg + b * kStgBytes + ((RO * cw) * kTX + xh * kCX) * kStgStride + (lane & 1) * 8;
            const int sc = lane >> 1;
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
                for (int r = 0; r < RO; ++r) *reinterpret_cast<float2*>(so + (r * kTX + x) * kStgStride + ((sc ^ x) << 4)) = acc[r];
            }
            mbar_arrive(&a_empty[s]);      // the V patch of this stage is no longer needed
            mbar_arrive(&conv_full[b]);
            // The conv warp that finishes a patch last counts it as applied (one arrival per patch and CTA: the state
            // pipelines poll these counters).  Warps are at most a few patches apart, far less than 8.
            if (lane == 0 && (atomicAdd(&applied_s[it & 7], 1u) % G::kConvWarps) == G::kConvWarps - 1)
                atomicAdd(plane_ctr + (size_t)bh * kPipeCtrPerPlane + kPipeCtrApplied, 1u);
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    // The CTA that leaves last puts the counters back to zero for the next call.
    if (tid == 0) {
        __threadfence();
        *last_slot = (atomicAdd(prm.ctr, 1u) == (unsigned)(n_cta - 1));
    }
    __syncthreads();
    if (*last_slot) {
        __threadfence();
        for (int i = tid; i < prm.BH * kPipeCtrPerPlane; i += blockDim.x) plane_ctr[i] = 0;
        if (tid < kPipeCtrHeader) prm.ctr[tid] = 0;
    }
}

template <int KS, int MODE>
cudaError_t launch_pipe_ks(const Problem& p, float* state, float* ready, unsigned* ctr, unsigned* status, cudaStream_t st) {
    constexpr bool PAIR = (MODE == 1);
    using G = PGeo<KS, PAIR>;
    const bool pair = PAIR;
    const int rows = pair ? p.N / 2 : p.N;            // 128-byte rows per plane (leading off-grid tokens included)
    const int cols = pair ? p.gridW / 2 : p.gridW;    // 128-byte columns per grid row
    const PipePlan plan = plan_pipe(p.BH, rows, cols, p.gridH);
    if (!plan.ok) return cudaErrorNotSupported;
    const uint64_t nb = (uint64_t)(p.BH / p.hdiv);
    CUtensorMap tmK, tmVs, tmQ, tmVh, tmO;
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
        uint64_t sq[4], sv[4], so[4];
        strides(p.lq, sq); strides(p.lv, sv); strides(p.lo, so);
        const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + p.prefix * p.lq.token;
        const __nv_bfloat16* vg = static_cast<const __nv_bfloat16*>(p.v) + p.prefix * p.lv.token;
        __nv_bfloat16* og = static_cast<__nv_bfloat16*>(p.out) + p.prefix * p.lo.token;
        if (!make_tensor_map_bf16(&tmQ, qg, rank, dims, sq, box, true) || !make_tensor_map_bf16(&tmVh, vg, rank, dims, sv, boxv, false) ||
            !make_tensor_map_bf16(&tmO, og, rank, dims, so, box, true))
            return cudaErrorNotSupported;
    }
    PipeParams prm;
    prm.state = state; prm.ready = ready; prm.ctr = ctr;
    prm.w = static_cast<const __nv_bfloat16*>(p.w);
    prm.bias = static_cast<const __nv_bfloat16*>(p.bias);
    prm.flat = (rank == 4) ? 1 : 0;
    prm.H = p.H; prm.head0 = p.head0; prm.BH = p.BH; prm.hdiv = p.hdiv;
    prm.tilesX = (cols + kTX - 1) / kTX; prm.tilesY = (p.gridH + kTY - 1) / kTY;
    prm.s_tiles = plan.s_tiles; prm.chunk_tiles = plan.chunk_tiles; prm.n_chunks = plan.n_chunks;
    prm.ahead = plan.ahead;
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
    return cudaLaunchKernelEx(&cfg, tc_pipe_kernel<KS, MODE>, tmK, tmVs, tmQ, tmVh, tmO, prm);
}

// Planes that the state pipeline may be ahead of the apply pipeline: as many as keep the V rows read and not
// yet applied within a part of L2 that the other streams leave alone.
int planes_ahead(int BH, int rows) {
    const long long budget = 40ll << 20;
    long long ahead = budget / ((long long)(rows < 1 ? 1 : rows) * 128);
    if (ahead < 2) ahead = 2;  // at least two: a CTA finishes plane p between two of its chunks, and the next may belong to plane p + 1
    return (int)(ahead < BH ? ahead : BH);
}

}  // namespace

// Work split of the one-kernel forward: the rows of a plane are cut into chunks of kChunkTiles 64-row tiles,
// the grid into patches; one CTA per multiprocessor, or fewer when there is less work than that.
constexpr int kChunkTiles = 8;

PipePlan plan_pipe(int BH, int rows, int cols, int gridH) {
    PipePlan pl = {};
    const int sms = device_sm_count();
    if (rows < 1 || BH < 1 || cols < 1 || gridH < 1) return pl;
    pl.s_tiles = (rows + kSTile - 1) / kSTile;
    pl.chunk_tiles = kChunkTiles;
    pl.n_chunks = (pl.s_tiles + kChunkTiles - 1) / kChunkTiles;
    const long long patches = (long long)BH * ((cols + kTX - 1) / kTX) * ((gridH + kTY - 1) / kTY);
    const long long chunks = (long long)BH * pl.n_chunks;
    const long long work = patches > chunks ? patches : chunks;
    pl.grid = (int)(work < sms ? work : sms);
    pl.ahead = planes_ahead(BH, rows);
    pl.ok = true;
    return pl;
}

size_t pipe_ready_words(int BH) { return (size_t)(BH < 0 ? 0 : BH) * kReadyWords; }

bool pipe_supports(const Problem& p) {
    const bool pair = (p.d == 32);
    return plan_pipe(p.BH, pair ? p.N / 2 : p.N, pair ? p.gridW / 2 : p.gridW, p.gridH).ok;
}

cudaError_t launch_pipe(const Problem& p, float* state, float* ready, unsigned* ctr, unsigned* status, cudaStream_t st) {
    if (p.d == 32)
        return p.ksize == 3 ? launch_pipe_ks<3, 1>(p, state, ready, ctr, status, st)
                            : launch_pipe_ks<5, 1>(p, state, ready, ctr, status, st);
    if (p.blockdiag)
        return p.ksize == 3 ? launch_pipe_ks<3, 2>(p, state, ready, ctr, status, st)
                            : launch_pipe_ks<5, 2>(p, state, ready, ctr, status, st);
    return p.ksize == 3 ? launch_pipe_ks<3, 0>(p, state, ready, ctr, status, st)
                        : launch_pipe_ks<5, 0>(p, state, ready, ctr, status, st);
}

}  // namespace tc
}  // namespace castling

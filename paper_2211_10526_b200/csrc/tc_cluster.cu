// Forward of the tensor-core path for planes of a few thousand rows, in ONE launch: a thread-block cluster per
// (b,h) plane (Eq. 9).  Every CTA of the cluster
//   1. builds the state of its share of the plane's 128-row tiles exactly as the state kernel does (K rows
//      normalised in place, S = K^^T V and s = sum V accumulated in TMEM) and leaves it in its shared memory;
//   2. after a cluster-wide arrival, adds up the states of all CTAs of the cluster, read through distributed
//      shared memory in rank order (fixed order: the result does not depend on timing), straight into the bf16
//      operand S / pi of the second contraction and the vector 1/2 s;
//   3. applies it to its share of the plane's 8 x 16 patches exactly as the apply kernel does
//      (out = q^ S / pi + 1/2 s + bias + DWConv(V)), reading V a second time from L2.
// No workspace, no second launch, no reduction through global memory.  Every CTA loads its own tiles (no
// multicast).  The waits on other CTAs are mbarrier waits with the same time limit as all others.
#include "tc_common.cuh"
#include "tc_host.cuh"

#include <atomic>
#include <cstdlib>

namespace castling {
namespace tc {
namespace {

constexpr int kD = 64;
constexpr int kWords = kD * kD + kD;
constexpr int kTY = 8, kTX = 16;
constexpr int kTile = kTY * kTX;
constexpr int kQBytes = kTile * kD * 2;
constexpr int kStgStride = kD * 4 + 16;
constexpr int kStgBytes = kTile * kStgStride;
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kTmemCols = 128;                // phase 1: two accumulation chains; phase 3: two accumulators
constexpr int kChains = 2;
constexpr int kMaxCluster = 8;                // portable cluster size limit
constexpr int kSTile = 128, kSTileBytes = kSTile * kD * 2, kSStageBytes = 2 * kSTileBytes;

template <int KS, bool PAIR> struct Geo {
    // ---- phase 3: geometry of the apply kernel ----
    static constexpr int kConvRows = (KS == 3) ? 2 : 4;
    static constexpr int kConvWarps = 2 * kTY / kConvRows, kConvThreads = kConvWarps * 32;
    static constexpr int kThreads = 64 + kEpiThreads + kConvThreads;
    static constexpr int R = KS / 2;
    static constexpr int HC = PAIR ? (R + 1) / 2 : R;
    static constexpr int HY = kTY + 2 * R, HX = kTX + 2 * HC;
    static constexpr int kVBytes = HY * HX * kD * 2;
    static constexpr int kStage = ((kQBytes + kVBytes + 1023) / 1024) * 1024;
    static constexpr int kStages = (KS == 3) ? 3 : 2;
    static constexpr int kOffS = 0, kOffOut = 8192, kOffStages = kOffOut + kQBytes;
    static constexpr int kOffStg = kOffStages + kStages * kStage;
    static constexpr int kOffRq = kOffStg + 2 * kStgBytes;
    static constexpr int kOffBar = kOffRq + 2 * kTile * 4;      // barriers (256 B), then 1/2 s + bias (256 B)
    static constexpr int kOffHs = kOffBar + 256;
    static constexpr size_t kSmem = 1024 + kOffHs + 256;
    // ---- phase 1: a ring of K|V stages over the front of the same memory; this CTA's state, the constant block
    //      of the first contraction and the phase's barriers sit in what becomes the staging area ----
    static constexpr int kSStages = kOffStg / kSStageBytes;      // 4 (3x3) or 3 (5x5)
    static constexpr int kOffPartial = kOffStg, kOffOnes = kOffPartial + 17 * 1024, kOffSBar = kOffOnes + 2048;  // ones: 1 KiB-aligned
    static constexpr int kNormGroups = (kThreads / 32 - 7) / 4;   // warps 7.. in groups of four
    static_assert(kSStages >= 2 && kOffSBar + 512 <= kOffRq && kWords * 4 <= 17 * 1024, "phase 1 fits");
};

struct ClusterParams {
    int C;                 // CTAs per cluster = per plane
    int tiles;             // 128-row tiles per plane
    const __nv_bfloat16* w;
    const __nv_bfloat16* bias;
    int flat;
    int H, head0, hdiv, tilesX, tilesY;
    float eps2;
    unsigned* status;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(kTryWaitSuspendNs)
        : "memory");
    return ok != 0;
}
// mbar_wait with cluster-scope acquire: the other CTAs' shared-memory writes before their arrival are visible.
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned* status,
                                                  unsigned bit) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicOr(status, bit);
                return false;
            }
        }
    }
}
__device__ __forceinline__ float4 ld_cluster4(uint32_t remote_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote_addr) : "memory");
    return v;
}
// All CTAs of the cluster have started and initialised their barriers (hardware cluster barrier, once).
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int KS, int MODE>
__global__ void __launch_bounds__((Geo<KS, MODE == 1>::kThreads), 1)
tc_cluster_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmVs,
                  const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmVh,
                  const __grid_constant__ CUtensorMap tmO, const ClusterParams prm) {
    constexpr bool PAIR = (MODE == 1), BLOCKDIAG = (MODE == 2), HALVES = (MODE != 0);
    using G = Geo<KS, PAIR>;
    constexpr int NS = G::kStages, SNS = G::kSStages, NG = G::kNormGroups;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // phase 3
    uint8_t* S_s = smem + G::kOffS;
    uint8_t* out_s = smem + G::kOffOut;
    uint8_t* stages = smem + G::kOffStages;
    uint8_t* stg = smem + G::kOffStg;
    float* rq_s = reinterpret_cast<float*>(smem + G::kOffRq);
    float* hs_s = reinterpret_cast<float*>(smem + G::kOffHs);            // token sums s (64 floats)
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + G::kOffBar);
    uint64_t* empty = full + NS;
    uint64_t* acc_full = empty + NS;
    uint64_t* conv_full = acc_full + 2;
    uint64_t* buf_free = conv_full + 2;
    uint64_t* cl_bar = buf_free + 2;                                     // arrivals of the cluster's CTAs
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(cl_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    // phase 1
    float* partial = reinterpret_cast<float*>(smem + G::kOffPartial);
    uint8_t* ones = smem + G::kOffOnes;
    uint64_t* sfull = reinterpret_cast<uint64_t*>(smem + G::kOffSBar);
    uint64_t* scaled = sfull + SNS;
    uint64_t* sempty = scaled + SNS;
    uint64_t* accum = sempty + SNS;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int C = prm.C;
    const int rank = (int)cluster_ctarank();
    const int bh = blockIdx.x / C;                       // the cluster's plane
    const int pb = bh / prm.hdiv, ph = bh - pb * prm.hdiv;
    const int t_begin = (int)((long long)prm.tiles * rank / C), t_end = (int)((long long)prm.tiles * (rank + 1) / C);
    const int n_tiles = t_end - t_begin;
    const int n_chains = n_tiles < kChains ? n_tiles : kChains;
    const int patches = prm.tilesX * prm.tilesY;
    const int my_tiles = rank < patches ? (patches - rank + C - 1) / C : 0;   // patches rank, rank + C, ...
    constexpr unsigned kBit = kStatusFusedTimeout;

    if (tid == 0) {
        for (int s = 0; s < SNS; ++s) { mbar_init(&sfull[s], 1); mbar_init(&scaled[s], kSTile); mbar_init(&sempty[s], 1); }
        mbar_init(accum, n_chains > 0 ? n_chains : 1);
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], G::kConvThreads + kEpiThreads + 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&conv_full[b], G::kConvThreads); mbar_init(&buf_free[b], kEpiThreads); }
        mbar_init(cl_bar, C);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmVs);
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmVh); tma_prefetch_desc(&tmO);
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    if (warp >= 2 && warp < 6) {
        const int t = tid - 64, r = t >> 3, ch = t & 7;
        uint4 val = make_uint4(0, 0, 0, 0);
        if ((ch ^ (r & 7)) == 0) val.x = 0x3f80u;
        *reinterpret_cast<uint4*>(ones + r * 128 + ch * 16) = val;
        fence_proxy_async_smem();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    cluster_sync_all();  // nobody arrives on a barrier that its owner has not initialised yet
    const uint32_t tmem = *tmem_slot;

    // =========================== phase 1: this CTA's share of the plane's state ===========================
    if (warp == 0) {
        if (lane == 0) {
            const uint64_t pol_k = l2_policy_evict_first(), pol_v = l2_policy_evict_last();
            int issued = 0;
            for (int t = t_begin; t < t_end; ++t, ++issued) {
                const int s = issued % SNS, use = issued / SNS;
                if (use > 0 && !mbar_wait(&sempty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) break;
                uint8_t* ks = smem + s * kSStageBytes;
                mbar_expect_tx(&sfull[s], kSStageBytes);
                tma_load_4d_hint(ks, &tmK, &sfull[s], 0, t * kSTile, ph, pb, pol_k);
                tma_load_4d_hint(ks + kSTileBytes, &tmVs, &sfull[s], 0, t * kSTile, ph, pb, pol_v);
            }
            if (*abort_flag) {
                for (int i = max(0, issued - SNS); i < issued; ++i)
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&sfull[i % SNS], (i / SNS) & 1); ++spin) {}
            }
        }
    } else if (warp == 1 || warp == 6) {
        // two accumulation chains, one issuing thread each: chain j takes tiles j, j + 2, ... into its own accumulator
        const int chain = (warp == 1) ? 0 : 1;
        if (lane == 0 && chain < n_chains) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, kD, true, true);
            const uint32_t ones_addr = smem_u32(ones);
            bool ok = true;
            for (int it = chain; it < n_tiles && ok; it += kChains) {
                const int s = it % SNS, use = it / SNS;
                ok = mbar_wait(&scaled[s], use & 1, abort_flag, prm.status, kBit);
                if (!ok) break;
                tcgen05_fence_after_sync();
                const uint32_t ka = smem_u32(smem + s * kSStageBytes), va = ka + kSTileBytes;
#pragma unroll
                for (int j = 0; j < kSTile / 16; ++j) {
                    const uint32_t a0 = ka + j * 2048, b0 = va + j * 2048;
                    const uint64_t a = umma_desc_sw128(a0, ones_addr - a0, 1024);
                    const uint64_t b = umma_desc_sw128(b0, 0, 1024);
                    umma_bf16(tmem + chain * kD, a, b, idesc, (it != chain || j != 0) ? 1u : 0u);
                }
                umma_commit(&sempty[s]);
            }
            if (ok) umma_commit(accum);
        }
    } else if (warp < 6) {
        // accumulators -> this CTA's state in shared memory (rows 0..63: S, row 64: s), where the cluster reads it
        const int quarter = warp & 3, row = quarter * 32 + lane;
        bool ok = true;
        if (n_chains > 0) ok = mbar_wait(accum, 0, abort_flag, prm.status, kBit);
        if (ok && quarter < 3) {
            tcgen05_fence_after_sync();
#pragma unroll
            for (int cc = 0; cc < kD / 16; ++cc) {
                float v[16], v1[16];
                if (n_chains > 0) {
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + cc * 16, v);
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + kD + cc * 16, v1);
                    tmem_ld_wait();
                }
                if (row <= kD) {
                    float4* o4 = reinterpret_cast<float4*>(partial + row * kD + cc * 16);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (n_chains > 0) o = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                        if (n_chains > 1) { o.x += v1[4 * e]; o.y += v1[4 * e + 1]; o.z += v1[4 * e + 2]; o.w += v1[4 * e + 3]; }
                        o4[e] = o;
                    }
                }
            }
            tcgen05_fence_before_sync();
        }
    } else {
        const int g = (warp - 7) >> 2, t = (tid - 224) & 127;
        if (g < NG) {
            for (int gt = g; gt < n_tiles; gt += NG) {
                const int s = gt % SNS, use = gt / SNS;
                if (!mbar_wait(&sfull[s], use & 1, abort_flag, prm.status, kBit)) break;
                uint8_t* row = smem + s * kSStageBytes + t * 128;
                uint4 cch[8];
                float ssa = 0.f, ssb = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    cch[j] = *reinterpret_cast<const uint4*>(row + ((j ^ (t & 7)) << 4));
                    const uint32_t w[4] = {cch[j].x, cch[j].y, cch[j].z, cch[j].w};
                    float part = 0.f;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float lo = bf16lo(w[e]), hi = bf16hi(w[e]);
                        part = fmaf(lo, lo, part);
                        part = fmaf(hi, hi, part);
                    }
                    if (j < 4) ssa += part; else ssb += part;
                }
                float rka, rkb;
                if (HALVES) {
                    rka = 1.0f / sqrtf(fmaxf(ssa, prm.eps2));
                    rkb = 1.0f / sqrtf(fmaxf(ssb, prm.eps2));
                } else {
                    rka = rkb = 1.0f / sqrtf(fmaxf(ssa + ssb, prm.eps2));
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float rk = j < 4 ? rka : rkb;
                    uint4 o;
                    o.x = pack_bf16x2(bf16lo(cch[j].x) * rk, bf16hi(cch[j].x) * rk);
                    o.y = pack_bf16x2(bf16lo(cch[j].y) * rk, bf16hi(cch[j].y) * rk);
                    o.z = pack_bf16x2(bf16lo(cch[j].z) * rk, bf16hi(cch[j].z) * rk);
                    o.w = pack_bf16x2(bf16lo(cch[j].w) * rk, bf16hi(cch[j].w) * rk);
                    *reinterpret_cast<uint4*>(row + ((j ^ (t & 7)) << 4)) = o;
                }
                fence_proxy_async_smem();
                mbar_arrive(&scaled[s]);
            }
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();   // this CTA's state is complete in `partial`; the ring and the accumulators are dead
    tcgen05_fence_after_sync();

    // =========================== phase 2: sum over the cluster, in rank order ===========================
    if (tid == 0) {
        asm volatile("fence.acq_rel.cluster;" ::: "memory");
        for (int r = 0; r < C; ++r) mbar_arrive_cluster(map_to_rank(smem_u32(cl_bar), (uint32_t)r));
    }
    bool alive = mbar_wait_cluster(cl_bar, 0, abort_flag, prm.status, kBit);
    if (alive) {
        const uint32_t part_addr = smem_u32(partial);
        auto sum4 = [&](int word) -> float4 {   // four consecutive state words, summed over the CTAs in rank order
            float4 v[kMaxCluster];                // every load is issued before the first addition
#pragma unroll
            for (int r = 0; r < kMaxCluster; ++r)
                v[r] = (r < C) ? ld_cluster4(map_to_rank(part_addr + word * 4, (uint32_t)r)) : make_float4(0.f, 0.f, 0.f, 0.f);
            float4 acc = v[0];
#pragma unroll
            for (int r = 1; r < kMaxCluster; ++r)
                if (r < C) { acc.x += v[r].x; acc.y += v[r].y; acc.z += v[r].z; acc.w += v[r].w; }
            return acc;
        };
        if (warp >= 2 && warp < 2 + kEpiWarps) {
            // S / pi as the bf16 operand of the second contraction (rows: key features, 128-byte swizzle)
            const int et = tid - 64, i = et >> 2, part = et & 3;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                float4 lo, hi;
                if (!PAIR) {
                    lo = sum4(i * kD + part * 16 + 8 * c);
                    hi = sum4(i * kD + part * 16 + 8 * c + 4);
                    if (BLOCKDIAG && ((i < 32) != (part < 2))) { lo = make_float4(0.f, 0.f, 0.f, 0.f); hi = lo; }
                } else {
                    const int col = part * 16 + c * 8;
                    if ((i < 32) == (col < 32)) {
                        const int aa = i & 31, bcol = col & 31;
                        const float4 l0 = sum4(aa * kD + bcol), h0 = sum4(aa * kD + bcol + 4);
                        const float4 l1 = sum4((32 + aa) * kD + 32 + bcol), h1 = sum4((32 + aa) * kD + 32 + bcol + 4);
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
        } else if (warp == 2 + kEpiWarps && lane < 16) {
            // token sums s: row 64 of the state
            *reinterpret_cast<float4*>(hs_s + lane * 4) = sum4(kD * kD + lane * 4);
        }
    }
    __syncthreads();   // S / pi and s are in place (or the CTA has given up)
    if (tid == 0) {
        // this CTA has finished reading the other CTAs' states: they may overwrite them (and leave) after all C arrivals
        for (int r = 0; r < C; ++r) mbar_arrive_cluster(map_to_rank(smem_u32(cl_bar), (uint32_t)r));
    }
    // Nobody overwrites the staging area (where `partial` lives) or leaves before every CTA has read it.  A CTA that
    // gave up still arrives above, so that the others are not held up by it.
    if (alive) alive = mbar_wait_cluster(cl_bar, 1, abort_flag, prm.status, kBit);
    else (void)mbar_wait_cluster(cl_bar, 1, abort_flag, prm.status, kBit);

    // =========================== phase 3: this CTA's patches (rank, rank + C, ...) ===========================
    if (alive && my_tiles > 0) {
        if (warp == 0) {
            if (lane == 0) {
                int issued = 0;
                const uint64_t pol_q = l2_policy_evict_first();
                for (int it = 0; it < my_tiles; ++it) {
                    const int s = it % NS, use = it / NS;
                    const int j = rank + it * C, py = j / prm.tilesX, px = j - py * prm.tilesX;
                    const int y0 = py * kTY, x0 = px * kTX;
                    if (use > 0 && !mbar_wait(&empty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) break;
                    uint8_t* qs = stages + s * G::kStage;
                    mbar_expect_tx(&full[s], kQBytes + G::kVBytes);
                    if (prm.flat) {
                        tma_load_4d_hint(qs, &tmQ, &full[s], 0, x0, y0, bh, pol_q);
                        tma_load_4d(qs + kQBytes, &tmVh, &full[s], 0, x0 - G::HC, y0 - G::R, bh);
                    } else {
                        tma_load_5d_hint(qs, &tmQ, &full[s], 0, x0, y0, ph, pb, pol_q);
                        tma_load_5d(qs + kQBytes, &tmVh, &full[s], 0, x0 - G::HC, y0 - G::R, ph, pb);
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
                constexpr uint32_t idesc = umma_idesc_bf16(128, kD, false, true);
                const uint32_t s_addr = smem_u32(S_s);
                for (int it = 0; it < my_tiles; ++it) {
                    const int s = it % NS, use = it / NS, b = it & 1, ub = it >> 1;
                    if (!mbar_wait(&full[s], use & 1, abort_flag, prm.status, kBit)) break;
                    if (ub > 0 && !mbar_wait(&buf_free[b], (ub - 1) & 1, abort_flag, prm.status, kBit)) break;
                    tcgen05_fence_after_sync();
                    const uint32_t q_addr = smem_u32(stages + s * G::kStage);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) {
                        const uint64_t ad = umma_desc_sw128(q_addr + k * 32, 0, 1024);
                        const uint64_t bd = umma_desc_sw128(s_addr + k * 2048, 0, 1024);
                        umma_bf16(tmem + b * kD, ad, bd, idesc, k != 0);
                    }
                    umma_commit(&acc_full[b]);
                    umma_commit(&empty[s]);
                }
            }
        } else if (warp < 2 + kEpiWarps) {
            const int quarter = warp & 3, row = quarter * 32 + lane, et = tid - 64;
            const int half = (warp - 2) >> 2;
            const bool leader = (et == 0);
            const uint64_t pol_o = l2_policy_evict_first();
            for (int it = 0; it < my_tiles; ++it) {
                const int b = it & 1, ub = it >> 1, s = it % NS, use = it / NS;
                const int j = rank + it * C, py = j / prm.tilesX, px = j - py * prm.tilesX;
                const int y0 = py * kTY, x0 = px * kTX;
                if (!mbar_wait(&full[s], use & 1, abort_flag, prm.status, kBit)) break;
                {
                    const uint8_t* qrow = stages + s * G::kStage + row * 128;
                    float ss[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        const uint4 cq = *reinterpret_cast<const uint4*>(qrow + (((4 * half + jj) ^ (row & 7)) << 4));
                        const uint32_t w4[4] = {cq.x, cq.y, cq.z, cq.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float lo = bf16lo(w4[e]), hi = bf16hi(w4[e]);
                            ss[e] = fmaf(lo, lo, ss[e]); ss[e] = fmaf(hi, hi, ss[e]);
                        }
                    }
                    rq_s[half * kTile + row] = (ss[0] + ss[1]) + (ss[2] + ss[3]);
                    mbar_arrive(&empty[s]);
                }
                if (!mbar_wait(&acc_full[b], ub & 1, abort_flag, prm.status, kBit)) break;
                tcgen05_fence_after_sync();
                float acc[32];
                {
                    float a0[16], a1[16];
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + b * kD + half * 32, a0);
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + b * kD + half * 32 + 16, a1);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e) { acc[e] = a0[e]; acc[16 + e] = a1[e]; }
                }
                if (!mbar_wait(&conv_full[b], ub & 1, abort_flag, prm.status, kBit)) break;
                if (it > 0 && leader) tma_store_wait_read();
                named_barrier_sync(1, kEpiThreads);
                const float rq = (PAIR || BLOCKDIAG)
                                     ? rsqrtf(fmaxf(rq_s[half * kTile + row], prm.eps2))
                                     : rsqrtf(fmaxf(rq_s[row] + rq_s[kTile + row], prm.eps2));
                const uint8_t* srow = stg + b * kStgBytes + row * kStgStride + half * 128;
                uint8_t* orow = out_s + row * 128;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float4 c0 = *reinterpret_cast<const float4*>(srow + e * 32);
                    const float4 c1 = *reinterpret_cast<const float4*>(srow + e * 32 + 16);
                    uint4 pk;
                    pk.x = pack_bf16x2(fmaf(acc[8 * e + 0], rq, c0.x), fmaf(acc[8 * e + 1], rq, c0.y));
                    pk.y = pack_bf16x2(fmaf(acc[8 * e + 2], rq, c0.z), fmaf(acc[8 * e + 3], rq, c0.w));
                    pk.z = pack_bf16x2(fmaf(acc[8 * e + 4], rq, c1.x), fmaf(acc[8 * e + 5], rq, c1.y));
                    pk.w = pack_bf16x2(fmaf(acc[8 * e + 6], rq, c1.z), fmaf(acc[8 * e + 7], rq, c1.w));
                    *reinterpret_cast<uint4*>(orow + (((half * 4 + e) ^ (row & 7)) << 4)) = pk;
                }
                tcgen05_fence_before_sync();
                mbar_arrive(&buf_free[b]);
                fence_proxy_async_smem();
                named_barrier_sync(1, kEpiThreads);
                if (leader) {
                    if (prm.flat) tma_store_4d_hint(&tmO, out_s, 0, x0, y0, bh, pol_o);
                    else tma_store_5d_hint(&tmO, out_s, 0, x0, y0, ph, pb, pol_o);
                    tma_store_commit();
                }
            }
            if (leader) tma_store_wait_all();
        } else {
            const int cw = (warp - 2 - kEpiWarps) >> 1, xh = (warp - 2 - kEpiWarps) & 1;
            constexpr int kCX = kTX / 2;
            constexpr int R = G::R, RO = G::kConvRows, ROWS = RO + 2 * R;
            float2 wreg[KS][KS];
            float2 cinit;
            {
                // this lane's channel pair: 2*lane of 64 channels, or (PAIR) 2*(lane & 15) of 32 channels
                const int cp2 = PAIR ? 2 * (lane & 15) : 2 * lane;
                const int ch = ((prm.head0 + bh) % prm.H) * (PAIR ? 32 : kD) + cp2;
                float s0, s1;
                if (PAIR) { s0 = hs_s[cp2] + hs_s[32 + cp2]; s1 = hs_s[cp2 + 1] + hs_s[32 + cp2 + 1]; }
                else { s0 = hs_s[cp2]; s1 = hs_s[cp2 + 1]; }
                cinit.x = 0.5f * s0; cinit.y = 0.5f * s1;
                if (prm.bias) { cinit.x += __bfloat162float(prm.bias[ch]); cinit.y += __bfloat162float(prm.bias[ch + 1]); }
#pragma unroll
                for (int dy = 0; dy < KS; ++dy)
#pragma unroll
                    for (int dx = 0; dx < KS; ++dx)
                        wreg[dy][dx] = make_float2(__bfloat162float(prm.w[(size_t)ch * KS * KS + dy * KS + dx]),
                                                   __bfloat162float(prm.w[(size_t)(ch + 1) * KS * KS + dy * KS + dx]));
            }
            for (int it = 0; it < my_tiles; ++it) {
                const int s = it % NS, use = it / NS, b = it & 1, ub = it >> 1;
                if (!mbar_wait(&full[s], use & 1, abort_flag, prm.status, kBit)) break;
                if (ub > 0 && !mbar_wait(&buf_free[b], (ub - 1) & 1, abort_flag, prm.status, kBit)) break;
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
                        const int t = STEP * x + KS - STEP + n;
#pragma unroll
                        for (int r = 0; r < ROWS; ++r) {
                            const uint32_t wv = *reinterpret_cast<const uint32_t*>(vh + r * G::HX * 128 + t * U);
                            win[r][t % KS] = make_float2(bf16lo(wv), bf16hi(wv));
                        }
                    }
                    float2 accv[RO];
#pragma unroll
                    for (int r = 0; r < RO; ++r) accv[r] = cinit;
#pragma unroll
                    for (int dy = 0; dy < KS; ++dy)
#pragma unroll
                        for (int dx = 0; dx < KS; ++dx)
#pragma unroll
                            for (int r = 0; r < RO; ++r)
                                accv[r] = ffma2(wreg[dy][dx], win[dy + r][(STEP * x + dx) % KS], accv[r]);
#pragma unroll
                    for (int r = 0; r < RO; ++r) *reinterpret_cast<float2*>(so + (r * kTX + x) * kStgStride) = accv[r];
                }
                mbar_arrive(&empty[s]);
                mbar_arrive(&conv_full[b]);
            }
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

template <int KS, int MODE>
cudaError_t launch_cluster_ks(const Problem& p, int C, unsigned* status, cudaStream_t st) {
    constexpr bool PAIR = (MODE == 1);
    using G = Geo<KS, PAIR>;
    const bool pair = (p.d == 32);
    const int rows = pair ? p.N / 2 : p.N;
    const int cols = PAIR ? p.gridW / 2 : p.gridW;
    const uint64_t nb = (uint64_t)(p.BH / p.hdiv);
    CUtensorMap tmK, tmVs, tmQ, tmVh, tmO;
    {   // phase 1: [64, rows, planes per batch step, batch steps]
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
    {   // phase 3: [64, columns, grid rows, planes per batch step, batch steps]
        const uint64_t dims[5] = {(uint64_t)kD, (uint64_t)cols, (uint64_t)p.gridH, (uint64_t)p.hdiv, nb};
        const uint32_t box[5] = {kD, kTX, kTY, 1, 1};
        const uint32_t boxv[5] = {kD, (uint32_t)G::HX, (uint32_t)G::HY, 1, 1};
        auto strides = [&](const Layout& l, uint64_t (&s)[4]) {
            s[0] = (uint64_t)(PAIR ? kD : l.token);
            s[1] = (uint64_t)(l.token * p.gridW);
            s[2] = (uint64_t)l.head;
            s[3] = (uint64_t)(nb > 1 ? l.batch : l.head * p.hdiv);
        };
        uint64_t sq[4], sv[4], so[4];
        strides(p.lq, sq); strides(p.lv, sv); strides(p.lo, so);
        if (!make_tensor_map_bf16(&tmQ, p.q, rank, dims, sq, box, true) || !make_tensor_map_bf16(&tmO, p.out, rank, dims, so, box, true) ||
            !make_tensor_map_bf16(&tmVh, p.v, rank, dims, sv, boxv, false))
            return cudaErrorNotSupported;
    }
    ClusterParams prm;
    prm.C = C; prm.tiles = (rows + kSTile - 1) / kSTile;
    prm.w = static_cast<const __nv_bfloat16*>(p.w);
    prm.bias = static_cast<const __nv_bfloat16*>(p.bias);
    prm.flat = (rank == 4) ? 1 : 0;
    prm.H = p.H; prm.head0 = p.head0; prm.hdiv = p.hdiv;
    prm.tilesX = (cols + kTX - 1) / kTX; prm.tilesY = (p.gridH + kTY - 1) / kTY;
    prm.eps2 = p.eps2; prm.status = status;
    static PerDevice opt_in;
    {
        const cudaError_t e = opt_in_smem(tc_cluster_kernel<KS, MODE>, G::kSmem, opt_in);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.BH * C)); cfg.blockDim = dim3(G::kThreads); cfg.dynamicSmemBytes = G::kSmem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc_cluster_kernel<KS, MODE>, tmK, tmVs, tmQ, tmVh, tmO, prm);
}

// Clusters of C CTAs of this instantiation that the device keeps resident at once (queried once per C).
template <int KS, int MODE>
int max_active_clusters(int C) {
    using G = Geo<KS, MODE == 1>;
    static std::atomic<int> cached[kMaxCluster + 1];
    const int have = cached[C].load(std::memory_order_relaxed);
    if (have != 0) return have;
    static PerDevice opt_in;
    if (opt_in_smem(tc_cluster_kernel<KS, MODE>, G::kSmem, opt_in) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)C); cfg.blockDim = dim3(G::kThreads); cfg.dynamicSmemBytes = G::kSmem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tc_cluster_kernel<KS, MODE>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    cached[C].store(n > 0 ? n : -1, std::memory_order_relaxed);
    return n > 0 ? n : -1;
}

int env_int(const char* name, int dflt) {
    const char* e = getenv(name);
    return (e && e[0]) ? atoi(e) : dflt;
}

}  // namespace

// CTAs per plane: the largest of 8, 4, 2 that keeps the whole launch resident at once (the device reports how many
// clusters of a size it holds) and gives every CTA at least one tile of rows and one patch; 0 when the shape is not for this kernel (planes that
// the single-CTA forward takes, planes too long for one launch to pay, leading tokens).
int cluster_size(const Problem& p) {
    if (!p.bf16 || (p.ksize != 3 && p.ksize != 5) || p.prefix != 0) return 0;
    const bool pair = (p.d == 32);
    const int rows = pair ? p.N / 2 : p.N, cols = pair ? p.gridW / 2 : p.gridW;
    const int tiles = (rows + kSTile - 1) / kSTile;
    const int patches = ((cols + kTX - 1) / kTX) * ((p.gridH + kTY - 1) / kTY);
    const int max_rows = env_int("CASTLING_TC_CLUSTER_MAX_ROWS", 16384);
    if (rows > max_rows) return 0;
    const int mode = p.d == 32 ? 1 : (p.blockdiag ? 2 : 0);
    for (int C = kMaxCluster; C >= 2; C >>= 1) {
        if (tiles < C || patches < C) continue;
        int fit;  // clusters of this size resident at once: the whole launch has to be one wave
        if (p.ksize == 3) fit = mode == 0 ? max_active_clusters<3, 0>(C) : mode == 1 ? max_active_clusters<3, 1>(C) : max_active_clusters<3, 2>(C);
        else fit = mode == 0 ? max_active_clusters<5, 0>(C) : mode == 1 ? max_active_clusters<5, 1>(C) : max_active_clusters<5, 2>(C);
        if (p.BH <= fit) return C;
    }
    return 0;
}

cudaError_t launch_cluster(const Problem& p, int C, unsigned* status, cudaStream_t st) {
    if (p.d == 32)
        return p.ksize == 3 ? launch_cluster_ks<3, 1>(p, C, status, st) : launch_cluster_ks<5, 1>(p, C, status, st);
    if (p.blockdiag)
        return p.ksize == 3 ? launch_cluster_ks<3, 2>(p, C, status, st) : launch_cluster_ks<5, 2>(p, C, status, st);
    return p.ksize == 3 ? launch_cluster_ks<3, 0>(p, C, status, st) : launch_cluster_ks<5, 0>(p, C, status, st);
}

}  // namespace tc
}  // namespace castling

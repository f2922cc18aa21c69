// Attention with the exact angular kernel (Eq. 4-5) on the tensor cores, bf16, head width 64:
//     out_t = sum_j (1 - arccos(q^_t . k^_j) / pi) v_j + bias + DWConv(V)_t
// with explicit weights, quadratic in the number of tokens.  A work item is a (plane, tile of 128 queries); for
// every tile of 128 keys of the plane
//   warp 0       TMA: K and V tiles (128-byte swizzle, rows beyond the plane zero-filled), the Q tile once per item
//   warps 2..5   scale every K row (and, once per item, every Q row) to a unit row in place, as bf16
//   warp 1       one thread issues the UMMAs: C[128 x 128] = Q^ K^^T into one of two TMEM buffers, and, one tile
//                behind, O[128 x 64] += W[128 x 128] V with the weights W from shared memory
//   warps 6..13  thread = (query, 64 of the 128 keys): cosines out of TMEM, clamp, 1 - arccos/pi (a polynomial in
//                |x| times sqrt(1 - |x|), Abramowitz & Stegun 4.4.45, |error| < 7e-5 rad: far below the bf16 rounding
//                of the weights), bf16 weights into the shared-memory operand of the second contraction
// and at the end of the item warps 6..9 (thread = query) read O, add bias and the depthwise convolution of V taken
// from global memory, and store the row.  Keys beyond the plane have k^ = 0, weight 1/2 and v = 0: no masking.
// With the auxiliary branch of training (Eq. 10) every item takes a first sweep over the keys that only forms the
// cosines and adds up exp(cosine) per query (keys beyond the plane excluded); in the second sweep the weight of a pair
// is the base weight (exact kernel, or its kept part 1/2 + x/pi) plus Mask_eps of its softmax probability.
// No workspace; every wait is bounded.
#include "tc_common.cuh"
#include "tc_host.cuh"

namespace castling {
namespace tc {
namespace {

constexpr int kD = 64;
constexpr int kTile = 128;
constexpr int kTileBytes = kTile * kD * 2;          // 16 KiB
constexpr int kStageBytes = 2 * kTileBytes;         // K then V
constexpr int kStages = 3;
constexpr int kPBytes = kTile * kTile * 2;          // weights of one tile pair: two 64-key blocks of 16 KiB
constexpr int kThreads = 14 * 32;
constexpr int kNormThreads = 128, kWThreads = 256;
constexpr int kTmemCols = 512;                      // cosines: 2 x 128 columns; output: 64 columns at 256
constexpr int kOffQ = 0, kOffStages = kTileBytes, kOffP = kOffStages + kStages * kStageBytes;
constexpr int kOffDen = kOffP + 2 * kPBytes;        // softmax denominators: one partial sum per weight thread
constexpr int kOffBar = kOffDen + 2 * kTile * 4;
constexpr size_t kSmem = 1024 + kOffBar + 256;
static_assert(kSmem <= 227 * 1024, "shared memory");

struct QuadParams {
    const __nv_bfloat16* v;      // for the convolution
    __nv_bfloat16* out;
    const __nv_bfloat16* w;
    const __nv_bfloat16* bias;
    Layout lv, lo;
    int hdiv, H, head0, BH, N, gridH, gridW, q_tiles, k_tiles, n_items;
    float eps2;
    unsigned* status;
    float sparse_eps;       // threshold of the mask (sparse sweeps only)
};

// 1 - arccos(x) / pi for x in [-1, 1]
__device__ __forceinline__ float angular_weight(float x) {
    const float ax = fminf(fabsf(x), 1.0f);
    const float t = 1.0f - ax;
    float p = fmaf(-0.0187293f, ax, 0.0742610f);
    p = fmaf(p, ax, -0.2121144f);
    p = fmaf(p, ax, 1.5707288f);
    const float ac = p * (t * rsqrtf(fmaxf(t, 1e-30f)));     // arccos(|x|)
    const float r = ac * kInvPi;                              // arccos(|x|) / pi
    return x >= 0.f ? 1.0f - r : r;                           // arccos(-a) = pi - arccos(a)
}

template <int KS, bool SPARSE, bool EXACT>
__global__ void __launch_bounds__(kThreads, 1)
tc_quad_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const QuadParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* Q_s = smem + kOffQ;
    uint8_t* stages = smem + kOffStages;
    uint8_t* P_s = smem + kOffP;
    float* den_s = reinterpret_cast<float*>(smem + kOffDen);
    uint64_t* q_full = reinterpret_cast<uint64_t*>(smem + kOffBar);
    uint64_t* q_ready = q_full + 1;      // Q rows scaled (128)
    uint64_t* q_free = q_ready + 1;      // the item's last cosine UMMAs have read Q
    uint64_t* kv_full = q_free + 1;      // [kStages]
    uint64_t* k_scaled = kv_full + kStages;
    uint64_t* kv_empty = k_scaled + kStages;
    uint64_t* c_full = kv_empty + kStages;   // [2]
    uint64_t* c_free = c_full + 2;           // [2] (256)
    uint64_t* p_full = c_free + 2;           // [2] (256)
    uint64_t* p_free = p_full + 2;           // [2]
    uint64_t* o_full = p_free + 2;
    uint64_t* o_free = o_full + 1;           // (128)
    uint64_t* den_bar = o_free + 1;          // (256) both halves of every query's denominator are in shared memory
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(den_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int my_items = ((int)blockIdx.x < prm.n_items) ? (prm.n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int KT = prm.k_tiles;
    const int sweeps = SPARSE ? 2 : 1;   // key tiles per item: sweeps * KT; the last sweep feeds the second contraction
    constexpr unsigned kBit = kStatusFusedTimeout;

    if (tid == 0) {
        mbar_init(q_full, 1); mbar_init(q_ready, kNormThreads); mbar_init(q_free, 1);
        for (int s = 0; s < kStages; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&k_scaled[s], kNormThreads); mbar_init(&kv_empty[s], 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&c_full[b], 1); mbar_init(&c_free[b], kWThreads); mbar_init(&p_full[b], kWThreads); mbar_init(&p_free[b], 1);
        }
        mbar_init(o_full, 1); mbar_init(o_free, kNormThreads); mbar_init(den_bar, kWThreads);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            long long g = 0;   // key tiles issued so far, over all items
            bool ok = true;
            for (int i = 0; i < my_items && ok; ++i) {
                const int item = blockIdx.x + i * gridDim.x, bh = item / prm.q_tiles, qt = item - bh * prm.q_tiles;
                const int pb = bh / prm.hdiv, ph = bh - pb * prm.hdiv;
                if (i > 0 && !mbar_wait(q_free, (i - 1) & 1, abort_flag, prm.status, kBit)) break;
                mbar_expect_tx(q_full, kTileBytes);
                tma_load_4d(Q_s, &tmQ, q_full, 0, qt * kTile, ph, pb);
                for (int tt = 0; tt < sweeps * KT; ++tt, ++g) {
                    const int jt = tt % KT;
                    const bool with_v = tt >= (sweeps - 1) * KT;   // the first sweep of two needs the keys only
                    const int s = (int)(g % kStages), use = (int)(g / kStages);
                    if (use > 0 && !mbar_wait(&kv_empty[s], (use - 1) & 1, abort_flag, prm.status, kBit)) { ok = false; break; }
                    uint8_t* ks = stages + s * kStageBytes;
                    mbar_expect_tx(&kv_full[s], with_v ? kStageBytes : kTileBytes);
                    tma_load_4d(ks, &tmK, &kv_full[s], 0, jt * kTile, ph, pb);
                    if (with_v) tma_load_4d(ks + kTileBytes, &tmV, &kv_full[s], 0, jt * kTile, ph, pb);
                }
            }
            if (*abort_flag) {  // giving up: let the copies in flight land before shared memory goes away
                for (long long i = (g > kStages ? g - kStages : 0); i < g; ++i)
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&kv_full[i % kStages], (uint32_t)((i / kStages) & 1)); ++spin) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_c = umma_idesc_bf16(128, 128, false, false);   // Q^ (K-major) x K^ (K-major)
            constexpr uint32_t idesc_o = umma_idesc_bf16(128, kD, false, true);     // W (K-major) x V (N-major)
            const uint32_t q_addr = smem_u32(Q_s), p_addr = smem_u32(P_s);
            long long g = 0, gp = 0;   // key tiles so far: all of them / those that feed the second contraction
            bool ok = true;
            // the second contraction of the tile with ring number gg and weight-buffer number pp; first: the item's first
            auto second = [&](long long gg, long long pp, bool first) -> bool {
                const int s = (int)(gg % kStages), pbuf = (int)(pp & 1);
                if (!mbar_wait(&p_full[pbuf], (uint32_t)((pp >> 1) & 1), abort_flag, prm.status, kBit)) return false;
                tcgen05_fence_after_sync();
                const uint32_t va = smem_u32(stages + s * kStageBytes + kTileBytes), pa = p_addr + pbuf * kPBytes;
#pragma unroll
                for (int j = 0; j < kTile / 16; ++j) {
                    const uint64_t a = umma_desc_sw128(pa + (j >> 2) * kTileBytes + (j & 3) * 32, 0, 1024);
                    const uint64_t b = umma_desc_sw128(va + j * 2048, 0, 1024);
                    umma_bf16(tmem + 256, a, b, idesc_o, (first && j == 0) ? 0u : 1u);
                }
                umma_commit(&p_free[pbuf]);
                umma_commit(&kv_empty[s]);
                return true;
            };
            for (int i = 0; i < my_items && ok; ++i) {
                if (!mbar_wait(q_ready, i & 1, abort_flag, prm.status, kBit)) break;
                // the previous item's output has been read out of TMEM before this item's first accumulation
                if (i > 0 && !mbar_wait(o_free, (i - 1) & 1, abort_flag, prm.status, kBit)) break;
                for (int tt = 0; tt < sweeps * KT && ok; ++tt, ++g) {
                    const bool last_sweep = tt >= (sweeps - 1) * KT;
                    const int jt = tt % KT;
                    const int s = (int)(g % kStages), use = (int)(g / kStages), cb = (int)(g & 1);
                    ok = mbar_wait(&k_scaled[s], use & 1, abort_flag, prm.status, kBit);
                    if (ok && g >= 2) ok = mbar_wait(&c_free[cb], (uint32_t)(((g >> 1) - 1) & 1), abort_flag, prm.status, kBit);
                    if (!ok) break;
                    tcgen05_fence_after_sync();
                    const uint32_t ka = smem_u32(stages + s * kStageBytes);
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) {
                        const uint64_t a = umma_desc_sw128(q_addr + k * 32, 0, 1024);
                        const uint64_t b = umma_desc_sw128(ka + k * 32, 0, 1024);
                        umma_bf16(tmem + cb * 128, a, b, idesc_c, k != 0);
                    }
                    umma_commit(&c_full[cb]);
                    if (!last_sweep) { umma_commit(&kv_empty[s]); continue; }   // cosines only: the stage is free again
                    if (jt == KT - 1) umma_commit(q_free);
                    if (jt > 0) { ok = second(g - 1, gp, jt == 1); ++gp; }   // one tile behind: the weight warps work meanwhile
                }
                if (ok) { ok = second(g - 1, gp, KT == 1); ++gp; }
                if (ok) umma_commit(o_full);
            }
        }
    } else if (warp < 6) {
        // ---- unit rows: Q once per item, K per tile ----
        const int t = tid - 64;
        auto scale_row = [&](uint8_t* row) {
            uint4 c[8];
            float ss = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                c[j] = *reinterpret_cast<const uint4*>(row + ((j ^ (t & 7)) << 4));
                const uint32_t w[4] = {c[j].x, c[j].y, c[j].z, c[j].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float lo = bf16lo(w[e]), hi = bf16hi(w[e]);
                    ss = fmaf(lo, lo, ss);
                    ss = fmaf(hi, hi, ss);
                }
            }
            const float rk = 1.0f / sqrtf(fmaxf(ss, prm.eps2));
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint4 o;
                o.x = pack_bf16x2(bf16lo(c[j].x) * rk, bf16hi(c[j].x) * rk);
                o.y = pack_bf16x2(bf16lo(c[j].y) * rk, bf16hi(c[j].y) * rk);
                o.z = pack_bf16x2(bf16lo(c[j].z) * rk, bf16hi(c[j].z) * rk);
                o.w = pack_bf16x2(bf16lo(c[j].w) * rk, bf16hi(c[j].w) * rk);
                *reinterpret_cast<uint4*>(row + ((j ^ (t & 7)) << 4)) = o;
            }
            fence_proxy_async_smem();
        };
        long long g = 0;
        bool ok = true;
        for (int i = 0; i < my_items && ok; ++i) {
            if (!mbar_wait(q_full, i & 1, abort_flag, prm.status, kBit)) break;
            scale_row(Q_s + t * 128);
            mbar_arrive(q_ready);
            for (int tt = 0; tt < sweeps * KT; ++tt, ++g) {
                const int s = (int)(g % kStages), use = (int)(g / kStages);
                if (!mbar_wait(&kv_full[s], use & 1, abort_flag, prm.status, kBit)) { ok = false; break; }
                scale_row(stages + s * kStageBytes + t * 128);
                mbar_arrive(&k_scaled[s]);
            }
        }
    } else {
        // ---- weights: thread = (query row, 64 of the tile's 128 keys); at the end of an item half 0 writes the rows ----
        const int quarter = warp & 3, half = (warp - 6) >> 2, row = quarter * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        long long g = 0, gp = 0;
        bool ok = true;
        for (int i = 0; i < my_items && ok; ++i) {
            const int item = blockIdx.x + i * gridDim.x, bh = item / prm.q_tiles, qt = item - bh * prm.q_tiles;
            float inv_den = 0.f;
            if (SPARSE) {
                // first sweep: sum over the plane's keys of exp(cosine) for this thread's query, half of every tile
                float den = 0.f;
                for (int jt = 0; jt < KT; ++jt, ++g) {
                    const int cb = (int)(g & 1);
                    if (!mbar_wait(&c_full[cb], (uint32_t)((g >> 1) & 1), abort_flag, prm.status, kBit)) { ok = false; break; }
                    tcgen05_fence_after_sync();
                    const int key0 = jt * kTile + half * 64;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        float x[16];
                        tmem_ld16(lane_base + cb * 128 + half * 64 + cc * 16, x);
                        tmem_ld_wait();
                        if (jt < KT - 1) {   // only the last tile can reach beyond the plane
#pragma unroll
                            for (int e = 0; e < 16; ++e) den += __expf(fminf(fmaxf(x[e], -1.0f), 1.0f));
                        } else {
#pragma unroll
                            for (int e = 0; e < 16; ++e)
                                if (key0 + cc * 16 + e < prm.N) den += __expf(fminf(fmaxf(x[e], -1.0f), 1.0f));
                        }
                    }
                    tcgen05_fence_before_sync();
                    mbar_arrive(&c_free[cb]);
                }
                if (!ok) break;
                den_s[half * kTile + row] = den;
                mbar_arrive(den_bar);
                if (!mbar_wait(den_bar, i & 1, abort_flag, prm.status, kBit)) break;
                inv_den = 1.0f / (den_s[row] + den_s[kTile + row]);
            }
            // weight of a pair from its cosine
            auto weight = [&](float xr) -> float {
                // rounding can leave a cosine just outside [-1, 1]; the exact kernel's function clamps |x| itself
                const float x = (EXACT && !SPARSE) ? xr : fminf(fmaxf(xr, -1.0f), 1.0f);
                float wv = EXACT ? angular_weight(x) : fmaf(x, kInvPi, 0.5f);
                if (SPARSE) {
                    const float pr = __expf(x) * inv_den;
                    if (pr > prm.sparse_eps) wv += pr;
                }
                return wv;
            };
            for (int jt = 0; jt < KT; ++jt, ++g, ++gp) {
                const int cb = (int)(g & 1), pbuf = (int)(gp & 1);
                if (!mbar_wait(&c_full[cb], (uint32_t)((g >> 1) & 1), abort_flag, prm.status, kBit)) { ok = false; break; }
                tcgen05_fence_after_sync();
                if (gp >= 2 && !mbar_wait(&p_free[pbuf], (uint32_t)(((gp >> 1) - 1) & 1), abort_flag, prm.status, kBit)) { ok = false; break; }
                uint8_t* prow = P_s + pbuf * kPBytes + half * kTileBytes + row * 128;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    float x[16];
                    tmem_ld16(lane_base + cb * 128 + half * 64 + cc * 16, x);
                    tmem_ld_wait();
                    uint4 o0, o1;
                    o0.x = pack_bf16x2(weight(x[0]), weight(x[1]));
                    o0.y = pack_bf16x2(weight(x[2]), weight(x[3]));
                    o0.z = pack_bf16x2(weight(x[4]), weight(x[5]));
                    o0.w = pack_bf16x2(weight(x[6]), weight(x[7]));
                    o1.x = pack_bf16x2(weight(x[8]), weight(x[9]));
                    o1.y = pack_bf16x2(weight(x[10]), weight(x[11]));
                    o1.z = pack_bf16x2(weight(x[12]), weight(x[13]));
                    o1.w = pack_bf16x2(weight(x[14]), weight(x[15]));
                    *reinterpret_cast<uint4*>(prow + (((2 * cc) ^ (row & 7)) << 4)) = o0;
                    *reinterpret_cast<uint4*>(prow + (((2 * cc + 1) ^ (row & 7)) << 4)) = o1;
                }
                tcgen05_fence_before_sync();
                mbar_arrive(&c_free[cb]);
                fence_proxy_async_smem();
                mbar_arrive(&p_full[pbuf]);
            }
            if (!ok) break;
            if (half == 0) {
                if (!mbar_wait(o_full, i & 1, abort_flag, prm.status, kBit)) break;
                tcgen05_fence_after_sync();
                float o[kD];
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    float x[16];
                    tmem_ld16(lane_base + 256 + cc * 16, x);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e) o[cc * 16 + e] = x[e];
                }
                tcgen05_fence_before_sync();
                mbar_arrive(o_free);
                const int tq = qt * kTile + row;
                if (tq < prm.N) {
                    const int y = tq / prm.gridW, xq = tq - y * prm.gridW;
                    constexpr int R = KS / 2;
                    const __nv_bfloat16* vp = prm.v + plane_offset(prm.lv, bh, prm.hdiv);
                    // filters and bias of the item's head: the same address in every lane (a broadcast from L1)
                    const int hh = (prm.head0 + bh) % prm.H;
                    const __nv_bfloat16* wh = prm.w + (size_t)hh * kD * (KS * KS);
                    if (prm.bias) {
#pragma unroll
                        for (int c = 0; c < kD; ++c) o[c] += __bfloat162float(prm.bias[hh * kD + c]);
                    }
                    for (int dy = 0; dy < KS; ++dy) {
                        const int yy = y + dy - R;
                        if ((unsigned)yy >= (unsigned)prm.gridH) continue;
                        for (int dx = 0; dx < KS; ++dx) {
                            const int xx = xq + dx - R;
                            if ((unsigned)xx >= (unsigned)prm.gridW) continue;
                            const uint4* vr = reinterpret_cast<const uint4*>(vp + (size_t)(yy * prm.gridW + xx) * prm.lv.token);
                            const __nv_bfloat16* fw = wh + dy * KS + dx;   // channel c at fw[c * KS * KS]
#pragma unroll
                            for (int c8 = 0; c8 < 8; ++c8) {
                                const uint4 vv = __ldg(vr + c8);
                                const uint32_t w4[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    o[c8 * 8 + 2 * e] = fmaf(__bfloat162float(fw[(c8 * 8 + 2 * e) * (KS * KS)]), bf16lo(w4[e]), o[c8 * 8 + 2 * e]);
                                    o[c8 * 8 + 2 * e + 1] = fmaf(__bfloat162float(fw[(c8 * 8 + 2 * e + 1) * (KS * KS)]), bf16hi(w4[e]), o[c8 * 8 + 2 * e + 1]);
                                }
                            }
                        }
                    }
                    uint4* orow = reinterpret_cast<uint4*>(prm.out + plane_offset(prm.lo, bh, prm.hdiv) + (size_t)tq * prm.lo.token);
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) {
                        uint4 pk;
                        pk.x = pack_bf16x2(o[c8 * 8 + 0], o[c8 * 8 + 1]); pk.y = pack_bf16x2(o[c8 * 8 + 2], o[c8 * 8 + 3]);
                        pk.z = pack_bf16x2(o[c8 * 8 + 4], o[c8 * 8 + 5]); pk.w = pack_bf16x2(o[c8 * 8 + 6], o[c8 * 8 + 7]);
                        orow[c8] = pk;
                    }
                }
            }
        }
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

template <int KS, bool SPARSE, bool EXACT>
cudaError_t launch_quad_ks(const Problem& p, unsigned* status, cudaStream_t st) {
    CUtensorMap tmQ, tmK, tmV;
    const uint64_t nb = (uint64_t)(p.BH / p.hdiv);
    const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)p.N, (uint64_t)p.hdiv, nb};
    const uint32_t box[4] = {kD, kTile, 1, 1};
    auto strides = [&](const Layout& l, uint64_t (&s)[3]) {
        s[0] = (uint64_t)l.token; s[1] = (uint64_t)l.head; s[2] = (uint64_t)(nb > 1 ? l.batch : l.head * p.hdiv);
    };
    uint64_t sq[3], sk[3], sv[3];
    strides(p.lq, sq); strides(p.lk, sk); strides(p.lv, sv);
    if (!make_tensor_map_bf16(&tmQ, p.q, 4, dims, sq, box, true) || !make_tensor_map_bf16(&tmK, p.k, 4, dims, sk, box, true) ||
        !make_tensor_map_bf16(&tmV, p.v, 4, dims, sv, box, true))
        return cudaErrorNotSupported;
    QuadParams prm;
    prm.v = static_cast<const __nv_bfloat16*>(p.v);
    prm.out = static_cast<__nv_bfloat16*>(p.out);
    prm.w = static_cast<const __nv_bfloat16*>(p.w);
    prm.bias = static_cast<const __nv_bfloat16*>(p.bias);
    prm.lv = p.lv; prm.lo = p.lo;
    prm.hdiv = p.hdiv; prm.H = p.H; prm.head0 = p.head0; prm.BH = p.BH; prm.N = p.N;
    prm.gridH = p.gridH; prm.gridW = p.gridW;
    prm.q_tiles = (p.N + kTile - 1) / kTile; prm.k_tiles = prm.q_tiles;
    prm.n_items = p.BH * prm.q_tiles;
    prm.eps2 = p.eps2; prm.status = status;
    prm.sparse_eps = p.sparse_eps;
    static PerDevice opt_in;
    {
        const cudaError_t e = opt_in_smem(tc_quad_kernel<KS, SPARSE, EXACT>, kSmem, opt_in);
        if (e != cudaSuccess) return e;
    }
    const int sms = device_sm_count();
    const int grid = prm.n_items < sms ? prm.n_items : sms;
    tc_quad_kernel<KS, SPARSE, EXACT><<<(unsigned)grid, kThreads, kSmem, st>>>(tmQ, tmK, tmV, prm);
    return cudaGetLastError();
}

}  // namespace

// bf16, head width 64 (16-byte aligned token rows), 3x3 or 5x5 filters, explicit weights (exact kernel and / or the
// masked softmax branch) without row-sum division, no leading tokens.
bool quad_supports(const Problem& p) {
    return p.bf16 && p.d == kD && (p.ksize == 3 || p.ksize == 5) && (p.exact_kernel || p.sparse) && !p.rownorm &&
           p.prefix == 0 && !p.blockdiag && (p.lv.token % 8) == 0 && (p.lo.token % 8) == 0;
}

cudaError_t launch_quad(const Problem& p, unsigned* status, cudaStream_t st) {
    if (p.sparse && p.exact_kernel)
        return p.ksize == 3 ? launch_quad_ks<3, true, true>(p, status, st) : launch_quad_ks<5, true, true>(p, status, st);
    if (p.sparse)
        return p.ksize == 3 ? launch_quad_ks<3, true, false>(p, status, st) : launch_quad_ks<5, true, false>(p, status, st);
    return p.ksize == 3 ? launch_quad_ks<3, false, true>(p, status, st) : launch_quad_ks<5, false, true>(p, status, st);
}

}  // namespace tc
}  // namespace castling

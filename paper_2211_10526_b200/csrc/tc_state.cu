// State kernel of the tensor-core path (bf16, d = 64): per (b,h) and token split,
//     S = sum_n k^_n^T v_n  (64 x 64)   and   s = sum_n v_n  (64)            (Eq. 9)
// as one tcgen05 contraction over tokens.  Per 128-token stage TMA brings the K and V tiles
// into 128-byte-swizzled shared memory; four warps scale every K row by 1 / max(||k||, eps) in
// place (the scale sits on the contracted index, so it cannot wait for an epilogue); one thread
// issues UMMAs with A = [K^ ; 1 0 0 ...] (128 x tokens, M-major: rows 0..63 are the key
// features, row 64 is all ones, which makes row 64 of the accumulator the token sum of V) and
// B = V (tokens x 64, N-major).  The fp32 accumulator lives in TMEM for the CTA's whole token
// range and is written once, as this split's partial state.
// RN (row-sum normalisation, Eq. 3's denominator on the kept kernel of Eq. 8) also needs sum_n k^_n: B gets a
// second 64-wide block along N from the same constant block ([V | 1 0 0 ...]), so column 64 of the accumulator is
// the row sum of A: rows 0..63 of it are sum_n k^_n, and the state has 64 more words.
#include "tc_common.cuh"
#include "tc_host.cuh"

namespace castling {
namespace tc {
namespace {

constexpr int kD = 64;
constexpr int kTile = 128;                   // tokens per stage
constexpr int kStages = 3;                  // 3 x 32 KiB: two CTAs fit on one SM
constexpr int kTileBytes = kTile * kD * 2;   // 16 KiB per operand tile
constexpr int kStageBytes = 2 * kTileBytes;  // K then V
constexpr int kOnesBytes = 2048;             // 16 token rows x 128 B: feature 64 = 1, 65..127 = 0
constexpr int kThreads = 192;                // warp 0 TMA, warp 1 UMMA, warps 2..5 scale + epilogue
constexpr int kTmemCols = 128;                // two 64-column accumulators: a CTA may serve several (b,h) (RN: twice that)
constexpr int kGroup = 4;                    // splits per first-level reduction group
constexpr size_t kSmemBytes = 1024 + kStages * kStageBytes + kOnesBytes + 256;

// PAIR = true serves head width 32: the [N][32] tensors are viewed as [N/2][64], one 128-byte row
// holding two consecutive tokens.  The same contraction then yields the four 32 x 32 blocks
// [k_even^T v_even, k_even^T v_odd; k_odd^T v_even, k_odd^T v_odd]; the state is the sum of the two
// diagonal blocks (and s the sum of the two halves of row 64), which the apply kernel folds when it
// reads them.  Each half row is normalised by its own token's norm.
// The same instantiation serves two width-32 heads stored side by side in one 128-byte row (head
// stride 32): identical arithmetic; there the consumers keep the two diagonal blocks apart, one per head.
template <bool PAIR, bool RN>
__global__ void __launch_bounds__(kThreads, 2)
tc_state_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                float* __restrict__ dst, float* __restrict__ final_state, unsigned* __restrict__ counters,
                int N, int tiles_per_cta, int P, int BH, int hdiv, int items_per_cta, float eps2, unsigned* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* ones = smem + kStages * kStageBytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(ones + kOnesBytes);  // TMA bytes landed
    uint64_t* scaled = full + kStages;                                // K rows normalised (128 arrivals)
    uint64_t* empty = scaled + kStages;                               // UMMAs of the stage retired
    uint64_t* accum = empty + kStages;                                // [2] whole accumulation of an item retired
    uint64_t* acc_free = accum + 2;                                   // [2] accumulator read out (128 arrivals)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_free + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    constexpr int kAcc = RN ? 2 * kD : kD;                 // accumulator columns
    constexpr int kStateW = kD * kD + kD + (RN ? kD : 0);  // words of one state: S, s, (RN) sum of the unit key rows
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Work items.  With P > 1 a CTA serves one (b,h, split).  With P == 1 (many heads, few tokens) a CTA
    // serves items_per_cta consecutive (b,h) one after another, so that barrier set-up, TMEM allocation
    // and the first load latency are paid once and the loads of the next (b,h) overlap the current one.
    const int total_tiles = (N + kTile - 1) / kTile;
    const int p = (P > 1) ? blockIdx.x % P : 0;
    const int bh0 = (P > 1) ? blockIdx.x / P : blockIdx.x * items_per_cta;
    const int n_items = (P > 1) ? 1 : min(items_per_cta, BH - bh0);
    const int t_begin = p * tiles_per_cta;
    const int n_tiles = min(total_tiles, t_begin + tiles_per_cta) - t_begin;  // per item
    const int bh = bh0;  // the (b,h) of the split reduction below (P > 1: the only item)
    if (n_tiles <= 0 || n_items <= 0) {  // the host never makes such a CTA; keep the partial well defined anyway
        pdl_wait_primary();
        if (P > 1) {
            float* out = dst + ((size_t)bh * P + p) * kStateW;
            for (int i = tid; i < kStateW; i += kThreads) out[i] = 0.f;
        }
        return;
    }

    pdl_launch_dependents();  // the apply kernel may begin its prologue while this grid drains
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&scaled[s], kTile);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(&accum[b], 1); mbar_init(&acc_free[b], kTile); }
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    if (warp == 1) tmem_alloc(tmem_slot, RN ? 2 * kTmemCols : kTmemCols);
    if (warp >= 2) {
        // constant block of A: for each of 16 token rows, element 64 (first of the second 64-wide
        // block along M) is 1.0 and the rest 0; 16-byte chunk c of row r sits at chunk c ^ (r & 7)
        const int t = tid - 64;  // 0..127 -> one 16-byte chunk each
        const int r = t >> 3, c = t & 7;
        uint4 val = make_uint4(0, 0, 0, 0);
        if ((c ^ (r & 7)) == 0) val.x = 0x3f80u;  // logical chunk 0: bf16 1.0 in its first element
        *reinterpret_cast<uint4*>(ones + r * 128 + c * 16) = val;
        fence_proxy_async_smem();
    }
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            // Both tensors stream through L2 once here.  V is read again by the apply kernel, but at long sequences it
            // does not survive until then whatever the hint, and lines marked evict-last pile up and slow the streams
            // of both kernels (measured: 132 -> 125 us per forward at 2 x 8 planes of 256 x 256 tokens).
            const uint64_t pol_k = l2_policy_evict_first(), pol_v = l2_policy_evict_first();
            bool ok = true;
            // Launched programmatically dependent on the kernel before it in the stream (the apply kernel of the
            // previous forward lets its dependents start early): everything above ran while that kernel drained.
            // Global memory is first touched here; the partial states and arrival counters are written only after
            // these loads have landed.
            pdl_wait_primary();
            for (int item = 0; item < n_items && ok; ++item) {
                for (int it = 0; it < n_tiles; ++it, ++issued) {
                    const int s = issued % kStages, use = issued / kStages;
                    if (use > 0 && !mbar_wait(&empty[s], (use - 1) & 1, abort_flag, status, kStatusStateTimeout)) { ok = false; break; }
                    uint8_t* ks = smem + s * kStageBytes;
                    mbar_expect_tx(&full[s], kStageBytes);
                    const int plane = bh0 + item, pb = plane / hdiv, ph = plane - pb * hdiv;
                    tma_load_4d_hint(ks, &tmK, &full[s], 0, (t_begin + it) * kTile, ph, pb, pol_k);
                    tma_load_4d_hint(ks + kTileBytes, &tmV, &full[s], 0, (t_begin + it) * kTile, ph, pb, pol_v);
                }
            }
            if (*abort_flag) {
                // giving up: let copies already in flight land before the CTA's shared memory goes away
                for (int i = max(0, issued - kStages); i < issued; ++i)
                    for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&full[i % kStages], (i / kStages) & 1); ++spin) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, kAcc, true, true);
            const uint32_t ones_addr = smem_u32(ones);
            bool ok = true;
            int gt = 0;  // tiles issued so far, over all items
            for (int item = 0; item < n_items && ok; ++item) {
                const int buf = item & 1;
                if (item >= 2) ok = mbar_wait(&acc_free[buf], ((item >> 1) - 1) & 1, abort_flag, status, kStatusStateTimeout);
                for (int it = 0; it < n_tiles && ok; ++it, ++gt) {
                    const int s = gt % kStages, use = gt / kStages;
                    ok = mbar_wait(&scaled[s], use & 1, abort_flag, status, kStatusStateTimeout);
                    if (!ok) break;
                    tcgen05_fence_after_sync();
                    const uint32_t ka = smem_u32(smem + s * kStageBytes), va = ka + kTileBytes;
#pragma unroll
                    for (int j = 0; j < kTile / 16; ++j) {  // one UMMA per 16 tokens (K = 16)
                        const uint32_t a0 = ka + j * 2048, b0 = va + j * 2048;
                        const uint64_t a = umma_desc_sw128(a0, ones_addr - a0, 1024);
                        const uint64_t b = umma_desc_sw128(b0, RN ? ones_addr - b0 : 0, 1024);
                        umma_bf16(tmem + buf * kAcc, a, b, idesc, (it | j) != 0);
                    }
                    umma_commit(&empty[s]);
                }
                if (ok) umma_commit(&accum[buf]);
            }
        }
    } else {
        const int t = tid - 64;  // token row of the stage handled by this thread
        const int quarter = warp & 3;
        bool ok = true;
        // read the finished accumulator of `item` out of TMEM: rows 0..63 are S, row 64 is s; a warp reads
        // TMEM lanes 32*(warp%4)..+31.  Runs one item late, so that the UMMAs of an item overlap the
        // normalisation of the next item's tiles.
        auto flush = [&](int item) -> bool {
            const int buf = item & 1;
            if (!mbar_wait(&accum[buf], (item >> 1) & 1, abort_flag, status, kStatusStateTimeout)) return false;
            tcgen05_fence_after_sync();
            if (quarter < 3) {
                float* out = dst + ((size_t)(bh0 + item) * P + p) * kStateW;
                const int row = quarter * 32 + lane;
#pragma unroll
                for (int cc = 0; cc < kD / 16; ++cc) {
                    float v[16];
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + buf * kAcc + cc * 16, v);
                    tmem_ld_wait();
                    if (row <= kD) {
                        float4* o4 = reinterpret_cast<float4*>(out + row * kD + cc * 16);  // row 64 lands on s
#pragma unroll
                        for (int e = 0; e < 4; ++e) o4[e] = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                    }
                }
                if (RN) {  // column 64: the row sums of A; rows 0..63 are sum_n k^_n, stored behind s
                    float v[16];
                    tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + buf * kAcc + kD, v);
                    tmem_ld_wait();
                    if (row < kD) out[kD * kD + kD + row] = v[0];
                }
            }
            tcgen05_fence_before_sync();
            mbar_arrive(&acc_free[buf]);
            return true;
        };
        int gt = 0;  // tiles handled so far, over all items
        for (int item = 0; item < n_items && ok; ++item) {
            for (int it = 0; it < n_tiles; ++it, ++gt) {
                const int s = gt % kStages, use = gt / kStages;
                ok = mbar_wait(&full[s], use & 1, abort_flag, status, kStatusStateTimeout);
                if (!ok) break;
                uint8_t* row = smem + s * kStageBytes + t * 128;
                uint4 c[8];
                float ssa = 0.f, ssb = 0.f;  // first / second half of the row (two tokens when PAIR)
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    c[j] = *reinterpret_cast<const uint4*>(row + ((j ^ (t & 7)) << 4));
                    const uint32_t w[4] = {c[j].x, c[j].y, c[j].z, c[j].w};
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
                if (PAIR) {
                    rka = 1.0f / sqrtf(fmaxf(ssa, eps2));
                    rkb = 1.0f / sqrtf(fmaxf(ssb, eps2));
                } else {
                    rka = rkb = 1.0f / sqrtf(fmaxf(ssa + ssb, eps2));
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float rk = j < 4 ? rka : rkb;
                    uint4 o;
                    o.x = pack_bf16x2(bf16lo(c[j].x) * rk, bf16hi(c[j].x) * rk);
                    o.y = pack_bf16x2(bf16lo(c[j].y) * rk, bf16hi(c[j].y) * rk);
                    o.z = pack_bf16x2(bf16lo(c[j].z) * rk, bf16hi(c[j].z) * rk);
                    o.w = pack_bf16x2(bf16lo(c[j].w) * rk, bf16hi(c[j].w) * rk);
                    *reinterpret_cast<uint4*>(row + ((j ^ (t & 7)) << 4)) = o;
                }
                fence_proxy_async_smem();
                mbar_arrive(&scaled[s]);
            }
            if (ok && item > 0) ok = flush(item - 1);
        }
        if (ok) ok = flush(n_items - 1);
    }
    tcgen05_fence_before_sync();
    __syncthreads();  // every thread's part of this split's partial state has been stored
    if (warp == 1) tmem_dealloc(tmem, RN ? 2 * kTmemCols : kTmemCols);

    // Cross-split reduction without a second launch and without any waiting, as a two-level tree
    // driven by arrival counters: the splits of a (b,h) form groups of kGroup; the CTA that arrives
    // last in its group sums the group's partial states in index order into the group's first slot,
    // then the group that arrives last sums the group results in index order into the final state.
    // The order of the additions is fixed, so the result does not depend on which CTAs came last.
    // Every counter is put back to zero by the CTA that consumed it.
    if (P > 1 && !*abort_flag) {
        __shared__ int is_last;
        constexpr int kWords = kStateW, kWords4 = kWords / 4, kIter = (kWords4 + kThreads - 1) / kThreads;
        unsigned* cnt = counters + (size_t)bh * kCountersPerHead;
        const int n_groups = (P + kGroup - 1) / kGroup, grp = p / kGroup;
        const int first = grp * kGroup, members = min(kGroup, P - first);
        float4* base = reinterpret_cast<float4*>(dst + (size_t)bh * P * kWords);
        // One thread publishes for the CTA: its device-wide fence after the CTA barrier covers the stores the other
        // threads made before that barrier; its fence after the atomic, followed by a CTA barrier, lets every thread
        // read what the other CTAs of the group published the same way.
        if (tid == 0) {
            __threadfence();
            is_last = (atomicAdd(&cnt[grp], 1u) == (unsigned)(members - 1));
            __threadfence();
        }
        __syncthreads();
        if (!is_last) return;
        // a single group (at most kGroup splits): its sum is the final state, no second level
        float4* fin = reinterpret_cast<float4*>(final_state + (size_t)bh * kWords);
        float4* level1 = (n_groups == 1) ? fin : base + (size_t)first * kWords4;
        if (members > 1) {
            float4 acc[kIter];
#pragma unroll
            for (int j = 0; j < kIter; ++j) {
                const int i = tid + j * kThreads;
                if (i < kWords4) acc[j] = __ldcg(base + (size_t)first * kWords4 + i);
            }
            // every load of the group is issued before the first addition (one trip to L2, not one per member);
            // the additions keep the members' order
            float4 v[kGroup - 1][kIter];
#pragma unroll
            for (int m = 1; m < kGroup; ++m)
#pragma unroll
                for (int j = 0; j < kIter; ++j) {
                    const int i = tid + j * kThreads;
                    v[m - 1][j] = (m < members && i < kWords4) ? __ldcg(base + (size_t)(first + m) * kWords4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
            for (int m = 1; m < kGroup; ++m)
#pragma unroll
                for (int j = 0; j < kIter; ++j) {
                    if (m < members) { acc[j].x += v[m - 1][j].x; acc[j].y += v[m - 1][j].y; acc[j].z += v[m - 1][j].z; acc[j].w += v[m - 1][j].w; }
                }
#pragma unroll
            for (int j = 0; j < kIter; ++j) {
                const int i = tid + j * kThreads;
                if (i < kWords4) level1[i] = acc[j];
            }
        }
        if (n_groups == 1) {
            if (tid == 0) cnt[grp] = 0;
            return;
        }
        __syncthreads();
        if (tid == 0) {
            cnt[grp] = 0;
            __threadfence();
            is_last = (atomicAdd(&cnt[kCountersPerHead - 1], 1u) == (unsigned)(n_groups - 1));
            __threadfence();
        }
        __syncthreads();
        if (!is_last) return;
        float4 acc[kIter];
#pragma unroll
        for (int j = 0; j < kIter; ++j) {
            const int i = tid + j * kThreads;
            if (i < kWords4) acc[j] = __ldcg(base + i);
        }
        for (int g0 = 1; g0 < n_groups; g0 += 4) {  // four groups per trip to L2, added in the groups' order
            float4 v[4][kIter];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int j = 0; j < kIter; ++j) {
                    const int i = tid + j * kThreads;
                    v[u][j] = (g0 + u < n_groups && i < kWords4) ? __ldcg(base + (size_t)(g0 + u) * kGroup * kWords4 + i)
                                                                  : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int j = 0; j < kIter; ++j) {
                    if (g0 + u < n_groups) { acc[j].x += v[u][j].x; acc[j].y += v[u][j].y; acc[j].z += v[u][j].z; acc[j].w += v[u][j].w; }
                }
        }
#pragma unroll
        for (int j = 0; j < kIter; ++j) {
            const int i = tid + j * kThreads;
            if (i < kWords4) fin[i] = acc[j];
        }
        if (tid == 0) cnt[kCountersPerHead - 1] = 0;
    }
}

}  // namespace

cudaError_t launch_state(const Problem& p, float* partial, float* final_state, unsigned* counters, int P,
                         int tiles_per_cta, unsigned* status, cudaStream_t st) {
    const bool pair = (p.d == 32);          // two tokens per 128-byte row
    const bool halves = pair || p.blockdiag;  // each half of a row has its own norm
    const int rows = pair ? p.N / 2 : p.N;  // 128-byte rows per (b,h)
    CUtensorMap tmK, tmV;
    // [64, rows, planes per batch step, batch steps]; a 128-byte row is one token, or two adjacent ones
    const uint64_t nb = (uint64_t)(p.BH / p.hdiv);
    const uint64_t dims[4] = {(uint64_t)kD, (uint64_t)rows, (uint64_t)p.hdiv, nb};
    const uint32_t box[4] = {kD, kTile, 1, 1};
    const uint64_t sk[3] = {(uint64_t)(pair ? kD : p.lk.token), (uint64_t)p.lk.head,
                            (uint64_t)(nb > 1 ? p.lk.batch : p.lk.head * p.hdiv)};
    const uint64_t sv[3] = {(uint64_t)(pair ? kD : p.lv.token), (uint64_t)p.lv.head,
                            (uint64_t)(nb > 1 ? p.lv.batch : p.lv.head * p.hdiv)};
    if (!make_tensor_map_bf16(&tmK, p.k, 4, dims, sk, box, true) || !make_tensor_map_bf16(&tmV, p.v, 4, dims, sv, box, true))
        return cudaErrorNotSupported;
    static PerDevice opt_in[4];
    {
        const cudaError_t e = p.rownorm ? (halves ? opt_in_smem(tc_state_kernel<true, true>, kSmemBytes, opt_in[3])
                                                  : opt_in_smem(tc_state_kernel<false, true>, kSmemBytes, opt_in[2]))
                                        : (halves ? opt_in_smem(tc_state_kernel<true, false>, kSmemBytes, opt_in[1])
                                                  : opt_in_smem(tc_state_kernel<false, false>, kSmemBytes, opt_in[0]));
        if (e != cudaSuccess) return e;
    }
    float* dst = P > 1 ? partial : final_state;
    // P == 1: a CTA serves several consecutive (b,h); at most two CTAs per multiprocessor so all are resident
    int grid = p.BH * P, items = 1;
    const int resident = 2 * device_sm_count();
    if (P == 1 && p.BH > resident) {
        items = (p.BH + resident - 1) / resident;
        grid = (p.BH + items - 1) / items;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    auto launch = [&](auto kernel) {
        return cudaLaunchKernelEx(&cfg, kernel, tmK, tmV, dst, final_state, counters, rows, tiles_per_cta, P, p.BH, p.hdiv, items,
                                  p.eps2, status);
    };
    if (p.rownorm) return halves ? launch(tc_state_kernel<true, true>) : launch(tc_state_kernel<false, true>);
    return halves ? launch(tc_state_kernel<true, false>) : launch(tc_state_kernel<false, false>);
}

}  // namespace tc
}  // namespace castling

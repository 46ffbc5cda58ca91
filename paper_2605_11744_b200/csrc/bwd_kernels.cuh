// Backward kernels (softmax VJP with the stop-gradient rule of Definition 3.2 / Lemma B.1):
//   bwd_rowdot_kernel   D_p = <dO_p, O_p>                                    (HBM-bound)
//   seg_attn_bwd_dq_kernel    dQ_p = scale * sum_{visible j} dS_pj K_j             (sg keys included)
//   seg_attn_bwd_dkv_kernel   dK_j = scale * sum_{diff(p,j)} dS_pj Q_p,  dV_j = sum_{diff(p,j)} P_pj dO_p
// with P = 2^(s*scale*log2e - LSE*log2e), dS = P * (dO V^T - D).  Both tensor-core kernels run
// 384 threads: warp 0 TMA producer, warp 1 tcgen05 issuer and TMEM owner, warps 4..11 element-wise
// work (warp w owns the 32 accumulator rows of TMEM lane quarter w % 4 and the column half
// (w - 4) / 4 of every 128-column tile; warps 2, 3 idle).  The element-wise work of a tile is cut in
// two phases - A: P from the scores, B: dS from P and dP - and the tensor-core issue order is
// arranged so that each phase runs while the tensor cores work on products that do not depend on
// it.  No atomics: a CTA owns its output tile, so results are bitwise reproducible.
#pragma once
#include <type_traits>

#include "mask.cuh"
#include "ptx.cuh"

namespace segattn {

constexpr int kBwdThreads = 384;
constexpr int kEwWarp0 = 4;   // first element-wise warp
constexpr int kEwWarps = 8;
constexpr float kLog2e = 1.4426950408889634f;
#ifndef SEGATTN_DKV_POLY_EVERY
#define SEGATTN_DKV_POLY_EVERY 1
#endif
#ifndef SEGATTN_DQ_POLY_EVERY
#define SEGATTN_DQ_POLY_EVERY 4
#endif
constexpr int kDqPolyEvery = SEGATTN_DQ_POLY_EVERY;     // every n-th pair of phase A's exponentials of the dQ pass; 0: none
constexpr int kDkvPolyEvery = SEGATTN_DKV_POLY_EVERY;   // 1: half of phase A's exponentials by polynomial, 2: a quarter; 0: none

// ------------------------------------------------------------------------------------------
// D[b][h][r] = sum_e dO[b][r][h][e] * O[b][r][h][e]; one group of D/8 threads per row, 16-byte loads,
// kRowdotUnroll rows per thread group with all their loads issued before the first is used (the kernel
// is a pure stream: what matters is the number of bytes in flight per SM).
constexpr int kRowdotUnroll = 4;
template <int D>
__global__ void __launch_bounds__(256) bwd_rowdot_kernel(const __nv_bfloat16* __restrict__ O,
                                                         const __nv_bfloat16* __restrict__ dO, float* __restrict__ Dvec,
                                                         int B, int Lq, int Hq, long long s0, long long s1,
                                                         long long s2) {
    constexpr int TPR = D / 8;          // threads per row
    constexpr int RPB = 256 / TPR;      // rows a block covers per pass
    const long long n_rows = (long long)B * Lq * Hq;
    const long long row0 = (long long)blockIdx.x * (RPB * kRowdotUnroll) + threadIdx.x / TPR;
    const int part = threadIdx.x % TPR;
    uint4 a[kRowdotUnroll], g[kRowdotUnroll];
    long long out[kRowdotUnroll];
#pragma unroll
    for (int u = 0; u < kRowdotUnroll; ++u) {
        const long long row = row0 + (long long)u * RPB;
        a[u] = make_uint4(0, 0, 0, 0);
        g[u] = a[u];
        out[u] = -1;
        if (row < n_rows) {
            int h, b, r;
            if (n_rows <= 0xffffffffLL) {   // 32-bit division is several times cheaper than 64-bit
                const unsigned bh = (unsigned)row / (unsigned)Hq;   // (b, r)
                h = (int)((unsigned)row - bh * (unsigned)Hq);
                b = (int)(bh / (unsigned)Lq);
                r = (int)(bh - (unsigned)b * (unsigned)Lq);
            } else {
                const long long bh = row / Hq;
                h = (int)(row - bh * Hq);
                b = (int)(bh / Lq);
                r = (int)(bh - (long long)b * Lq);
            }
            const long long off = b * s0 + (long long)r * s1 + h * s2 + part * 8;
            a[u] = *reinterpret_cast<const uint4*>(O + off);
            g[u] = *reinterpret_cast<const uint4*>(dO + off);
            out[u] = ((long long)b * Hq + h) * Lq + r;
        }
    }
#pragma unroll
    for (int u = 0; u < kRowdotUnroll; ++u) {
        const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a[u]);
        const __nv_bfloat162* pg = reinterpret_cast<const __nv_bfloat162*>(&g[u]);
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 x = __bfloat1622float2(pa[i]), y = __bfloat1622float2(pg[i]);
            acc = fmaf(x.x, y.x, acc);
            acc = fmaf(x.y, y.y, acc);
        }
#pragma unroll
        for (int o = TPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (out[u] >= 0 && part == 0) Dvec[out[u]] = acc;
    }
}

// ------------------------------------------------------------------------------------------
// Shared pieces of the two tensor-core kernels.

// One arrival per element-wise warp: every lane has fenced its tensor-memory accesses, the warp
// converges, one lane arrives.
__device__ __forceinline__ void ew_warp_arrive(uint32_t bar, int lane) {
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
}
__device__ __forceinline__ void ew_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// TMEM column of the bf16 A operand for K-step k (16 elements = 8 packed columns): the two
// column halves keep their packed values at the start of their own 64-column half, so that a
// warp never writes over fp32 columns the other half's warp may still have to read.
__device__ __forceinline__ uint32_t packed_a_col(int k) { return (uint32_t)((k >> 2) * 64 + (k & 3) * 8); }

// ------------------------------------------------------------------------------------------
// dQ pass.  TMEM (512 columns): S at [0,128) and [128,256) (alternating key tiles; dS, bf16, is
// written over the start of each half of the tile's S buffer), dP at [256,384), dQ accumulator at
// [384,384+D).  Tensor-core order per key tile j, one straight run once dS(j) is there:
// dP(j+1) | dQ(j) | S(j+2);  element-wise: A(j+1) runs meanwhile, B(j+1) as soon as dP(j+1) is done.
template <int D>
struct DqSmem {
    static constexpr int kPanels = D / 64;
    static constexpr uint32_t kTileBytes = kTile * D * 2;
    static constexpr int kKStages = 3;
    static constexpr int kVStages = 2;
    static constexpr uint32_t kQ = 0;
    static constexpr uint32_t kDO = kTileBytes;
    static constexpr uint32_t kK = 2 * kTileBytes;
    static constexpr uint32_t kV = kK + kKStages * kTileBytes;
    static constexpr uint32_t kTotal = kV + kVStages * kTileBytes;
    static constexpr uint32_t kDynamic = kTotal + 1024;
};

using DqItem = WorkItem;
__device__ __forceinline__ DqItem dq_decode(const BwdParams& prm, int idx) { return decode_item(prm, idx); }

// first visible key tile and number of visible key tiles of a work item of the dQ pass
__device__ __forceinline__ void dq_item_tiles(const BwdParams& prm, const DqItem& it, int* t_lo, int* n_tiles) {
    long long jl_lo, jl_hi;
    q_tile_kv_range(prm.geom, it.qt * kTile, it.cls, false, &jl_lo, &jl_hi);
    *t_lo = (int)(jl_lo / kTile);
    *n_tiles = jl_hi >= jl_lo ? (int)(jl_hi / kTile) - *t_lo + 1 : 0;
}

// Persistent: one CTA per SM walks the work list (one 128-row query tile of one (batch, query head)
// per item, heaviest first, dealt round-robin); the rings of K and V tiles and all phase counters
// run on across items, so that the next item's tiles arrive and its first products are issued
// while the element-wise warps finish the current one.
template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1) seg_attn_bwd_dq_kernel(const __grid_constant__ BwdParams prm) {
    using SM = DqSmem<D>;
    constexpr int trace_id = 1;
    (void)trace_id;
    TRACE_INIT();
    constexpr int NK = SM::kKStages, NV = SM::kVStages;
    enum { kBarQFull = 0, kBarQEmpty, kBarDoFull, kBarDoEmpty, kBarKFull, kBarKEmpty = kBarKFull + NK,
           kBarVFull = kBarKEmpty + NK, kBarVEmpty = kBarVFull + NV, kBarSFull = kBarVEmpty + NV, kBarDpFull = kBarSFull + 2,
           kBarDsFull, kBarDqFull, kNumBars };
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[kNumBars];
    __shared__ uint32_t tmem_slot;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + SM::kQ, sDO = smem_base + SM::kDO;
    auto sK = [&](int s) { return smem_base + SM::kK + s * SM::kTileBytes; };
    auto sV = [&](int s) { return smem_base + SM::kV + s * SM::kTileBytes; };
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    const MaskGeom& geo = prm.geom;

    if (tid == 0) {
        for (int i = 0; i < kNumBars; ++i) mbar_init(bar(i), i == kBarDsFull ? kEwWarps : 1);
        fence_mbar_init();
        prefetch_tmap(&prm.tq);
        prefetch_tmap(&prm.tk);
        prefetch_tmap(&prm.tv);
        prefetch_tmap(&prm.tdo);
    }
    __syncwarp();
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const uint32_t tS0 = tmem, tDp = tmem + 256, tDq = tmem + 384;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int qn = 0;       // work items with visible tiles started so far
            int g = 0;  // key tiles requested so far (all work items; far fewer than 2^31)
            bool ok = true;
            ItemWalk walk(blockIdx.x, gridDim.x, prm.n_items_dq);
        for (int item; ok && walk.next(&item);) {
                const DqItem it = dq_decode(prm, item);
                int t_lo, n;
                dq_item_tiles(prm, it, &t_lo, &n);
                if (n == 0) continue;
                const int r0 = it.qt * kTile;
                // Q is free once the previous item's last S is done; dO once the previous item's dQ, staged in
                // the dO buffer, has been stored
                if (!(ok = mbar_wait(bar(kBarQEmpty), (qn & 1) ^ 1, 11))) break;
                mbar_expect_tx(bar(kBarQFull), SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                    tma_load_4d(sQ + pnl * 16384, &prm.tq, bar(kBarQFull), pnl * 64, it.hq, r0, it.b);
                if (!(ok = mbar_wait(bar(kBarDoEmpty), (qn & 1) ^ 1, 12))) break;
                mbar_expect_tx(bar(kBarDoFull), SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                    tma_load_4d(sDO + pnl * 16384, &prm.tdo, bar(kBarDoFull), pnl * 64, it.hq, r0, it.b);
                ++qn;
                for (int j = 0; ok && j < n; ++j) {
                    const int gj = g + j;
                    const int sk = (int)(gj % NK), sv = (int)(gj % NV);
                    const int row = (t_lo + j) * kTile;
                    if (!(ok = mbar_wait(bar(kBarKEmpty + sk), (uint32_t)((gj / NK) & 1) ^ 1, 11))) break;
                    mbar_expect_tx(bar(kBarKFull + sk), SM::kTileBytes);
                    for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                        tma_load_4d(sK(sk) + pnl * 16384, &prm.tk, bar(kBarKFull + sk), pnl * 64, it.slot, row, it.b);
                    if (!(ok = mbar_wait(bar(kBarVEmpty + sv), (uint32_t)((gj / NV) & 1) ^ 1, 12))) break;
                    mbar_expect_tx(bar(kBarVFull + sv), SM::kTileBytes);
                    for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                        tma_load_4d(sV(sv) + pnl * 16384, &prm.tv, bar(kBarVFull + sv), pnl * 64, it.slot, row, it.b);
                }
                g += n;
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (whole warp, uniform control flow; one elected lane issues) ----------------
        constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
        constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, 0, 1);
        int qn = 0;
        int g = 0;  // key tiles of earlier work items (a CTA sees far fewer than 2^31)
        bool ok = true;
        ItemWalk walk(blockIdx.x, gridDim.x, prm.n_items_dq);
        for (int item; ok && walk.next(&item);) {
            const DqItem it = dq_decode(prm, item);
            int t_lo, n;
            dq_item_tiles(prm, it, &t_lo, &n);
            if (n == 0) continue;
            // Waits on tiles brought by TMA need no tcgen05 fence.
            auto wait_k = [&](int j) { return warp_wait(bar(kBarKFull + (g + j) % NK), (uint32_t)((g + j) / NK) & 1, 14); };
            auto wait_v = [&](int j) { return warp_wait(bar(kBarVFull + (g + j) % NV), (uint32_t)((g + j) / NV) & 1, 15); };
            auto issue_s = [&](int j) {   // S(j) = Q K_j^T into the S buffer of the tile's global parity
                const int gj = g + j;
                const uint64_t qd = make_sdesc(sQ, 16, 1024), kd = make_sdesc(sK(gj % NK), 16, 1024);
                const uint32_t d_s = tS0 + (uint32_t)(gj & 1) * 128;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = ((k / 4) * 16384 + (k % 4) * 32) >> 4;  // descriptor addresses count 16-byte units
                    mma_ss(d_s, qd + off, kd + off, idesc_s, k > 0);
                }
                mma_commit(bar(kBarSFull + (gj & 1)));
                mma_commit_if(j == n - 1, bar(kBarQEmpty));   // the item's last scores release Q
            };
            auto issue_dp = [&](int j) {  // dP(j) = dO V_j^T
                const int sv = (g + j) % NV;
                const uint64_t od = make_sdesc(sDO, 16, 1024), vd = make_sdesc(sV(sv), 16, 1024);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = ((k / 4) * 16384 + (k % 4) * 32) >> 4;
                    mma_ss(tDp, od + off, vd + off, idesc_s, k > 0);
                }
                mma_commit(bar(kBarVEmpty + sv));
                mma_commit(bar(kBarDpFull));
            };
            ok = warp_wait2(bar(kBarQFull), qn & 1, bar(kBarKFull + g % NK), (uint32_t)(g / NK) & 1, 13);
            if (ok) issue_s(0);
            ok = ok && warp_wait2(bar(kBarDoFull), qn & 1, bar(kBarVFull + g % NV), (uint32_t)(g / NV) & 1, 13);
            if (ok) issue_dp(0);
            if (ok && n > 1 && (ok = wait_k(1))) issue_s(1);
            // The loop is bound by the latency of its own control flow between the batches of products:
            // what a run needs at its start is polled together (one vote, one branch when all of it is
            // there, as it usually is), and optional completion signals are predicated.
            for (int j = 0; ok && j < n; ++j) {
                const int gj = g + j;
                const bool has1 = j + 1 < n;
                // V(j+1) landed (if there is one); dS(j) written and dP(j) read
                const bool ready = (!has1 | mbar_test_wait(bar(kBarVFull + (gj + 1) % NV), (uint32_t)((gj + 1) / NV) & 1)) &
                                   mbar_test_wait(bar(kBarDsFull), (uint32_t)(gj & 1));
                if (!__all_sync(0xffffffffu, ready)) {
                    ok = (!has1 || wait_v(j + 1)) && warp_wait(bar(kBarDsFull), (uint32_t)(gj & 1), 16);
                    if (!ok) break;
                }
                tc_fence_after();
                TRACE(lane == 0, j * 16 + 4);
                if (has1) issue_dp(j + 1);   // first: phase B of the next tile waits for it
                const int sk = gj % NK;
                const uint32_t a_ds = tS0 + (uint32_t)(gj & 1) * 128;
                const uint64_t kd = make_sdesc(sK(sk), 16384, 1024);
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k)
                    mma_ts(tDq, a_ds + packed_a_col(k), kd + ((k * 2048) >> 4), idesc_dq, (j > 0) || (k > 0));
                mma_commit(bar(kBarKEmpty + sk));
                mma_commit_if(j == n - 1, bar(kBarDqFull));
                // K(j+2) reuses the stage dQ(j-1) released one run ago: its load gets the first two products
                // of this run as extra time before it is waited for
                if (j + 2 < n && (ok = wait_k(j + 2))) issue_s(j + 2);    // overwrites dS(j): after dQ(j)
                TRACE(lane == 0, j * 16 + 5);
            }
            ++qn;
            g += n;
        }
    } else if (warp >= kEwWarp0) {
        // ---------------- element-wise: thread = query row, 64 of the tile's 128 key columns ----------------
        const int quarter = warp & 3, half = (warp - kEwWarp0) >> 2;
        const int row = 32 * quarter + lane;
        const uint32_t lane_off = (uint32_t)(32 * quarter) << 16;
        const uint32_t col_off = (uint32_t)half * 64;
        const float sl2 = prm.scale_log2;
        const uint64_t sl2x2 = f32x2(sl2, sl2);
        constexpr int DH = D / 2;  // this thread's share of the row
        int qn = 0;
        int g = 0;  // key tiles of earlier work items
        bool ok = true;
        ItemWalk walk(blockIdx.x, gridDim.x, prm.n_items_dq);
        for (int item; ok && walk.next(&item);) {
            const DqItem it = dq_decode(prm, item);
            int t_lo, n_tiles;
            dq_item_tiles(prm, it, &t_lo, &n_tiles);
            const int r0 = it.qt * kTile;
            const int r = r0 + row;
            const long long p = (long long)geo.q_pos0 + r;
            long long vlo_ll = lo_visible(geo, p, it.cls) - geo.kv_pos0;
            long long vhi_ll = p - geo.kv_pos0;
            if (vlo_ll < 0) vlo_ll = 0;
            if (vhi_ll > geo.kv_len - 1) vhi_ll = geo.kv_len - 1;
            const int vlo = (int)vlo_ll, vhi = (int)vhi_ll;
            long long full_lo = lo_visible(geo, (long long)geo.q_pos0 + r0 + kTile - 1, it.cls) - geo.kv_pos0;
            long long full_hi = (long long)geo.q_pos0 + r0 - geo.kv_pos0;
            if (full_hi > geo.kv_len - 1) full_hi = geo.kv_len - 1;
            const bool row_ok = r < geo.Lq;
            const long long sidx = ((long long)it.b * prm.Hq + it.hq) * geo.Lq + r;
            float lse2 = INFINITY, dsum = 0.f;  // +inf: an absent or keyless row gives P = 0
            if (row_ok) {
                const float l = prm.LSE[sidx];
                lse2 = (l == -INFINITY) ? INFINITY : l * kLog2e;
                dsum = prm.Dvec[sidx];
            }
            const uint64_t nlse2 = f32x2(-lse2, -lse2);
            const uint64_t ndsum2 = f32x2(-dsum, -dsum);
            float P[64];
            // phase A: P = 2^(S*scale*log2e - LSE*log2e) for this thread's 64 columns of S buffer `tS`
            auto phase_a = [&](auto masked_c, const uint32_t tS, const int c0) {
                constexpr bool MASKED = decltype(masked_c)::value;
                uint32_t sa_[32], sb_[32];
                tmem_ld_x32(tS + lane_off + col_off, sa_);
                tmem_ld_x32(tS + lane_off + col_off + 32, sb_);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t(&sv)[32] = c ? sb_ : sa_;
                    tmem_wait_ld_dep(sv);
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const uint64_t x01 = fma_f32x2(f32x2_bits(sv[i], sv[i + 1]), sl2x2, nlse2);
                        float p0, p1;
                        if (kDqPolyEvery > 0 && (i / 2) % (kDqPolyEvery > 0 ? kDqPolyEvery : 1) == 0) {
                            ex2_poly_x2(x01, p0, p1);
                        } else {
                            float t0, t1;
                            f32x2_unpack(x01, t0, t1);
                            p0 = ex2(t0);
                            p1 = ex2(t1);
                        }
                        if (MASKED) {
                            const int col = c0 + (int)col_off + c * 32 + i;
                            p0 = (col >= vlo && col <= vhi) ? p0 : 0.f;
                            p1 = (col + 1 >= vlo && col + 1 <= vhi) ? p1 : 0.f;
                        }
                        P[c * 32 + i] = p0;
                        P[c * 32 + i + 1] = p1;
                    }
                }
            };
            // phase B: dS = P * (dP - D), rounded to bf16, written over the start of this half of the tile's S
            // buffer (its scores went into P in phase A; the next product into that buffer is issued after dQ)
            auto phase_b = [&](const uint32_t tS) {
                uint32_t da_[32], db_[32];
                tmem_ld_x32(tDp + lane_off + col_off, da_);
                tmem_ld_x32(tDp + lane_off + col_off + 32, db_);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t(&dv)[32] = c ? db_ : da_;
                    tmem_wait_ld_dep(dv);
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const uint64_t ds2 = mul_f32x2(f32x2(P[c * 32 + i], P[c * 32 + i + 1]),
                                                       add_f32x2(f32x2_bits(dv[i], dv[i + 1]), ndsum2));
                        float d0, d1;
                        f32x2_unpack(ds2, d0, d1);
                        pk[i / 2] = pack_bf16(d0, d1);
                    }
                    tmem_st_x16(tS + lane_off + col_off + c * 16, pk);
                }
            };
            for (int j = 0; j < n_tiles; ++j) {
                const int gj = g + j;
                const uint32_t tS = tS0 + (uint32_t)(gj & 1) * 128;
                const int c0 = (t_lo + j) * kTile;
                const bool masked = !(c0 >= full_lo && c0 + kTile - 1 <= full_hi);
                ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull + (int)(gj & 1)), (uint32_t)((gj >> 1) & 1), 17));
                if (!ok) break;
                tc_fence_after();
                TRACE(tid == 128, j * 16 + 0);
                if (masked) phase_a(std::true_type{}, tS, c0);
                else phase_a(std::false_type{}, tS, c0);
                TRACE(tid == 128, j * 16 + 1);
                ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarDpFull), (uint32_t)(gj & 1), 19));
                if (!ok) break;
                tc_fence_after();
                TRACE(tid == 128, j * 16 + 2);
                phase_b(tS);
                tmem_wait_st();
                ew_warp_arrive(bar(kBarDsFull), lane);
                TRACE(tid == 128, j * 16 + 3);
            }
            if (!ok) break;
            if (n_tiles > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarDqFull), (uint32_t)(qn & 1), 18));
                if (!ok) break;
                tc_fence_after();
                ++qn;
            }
            __nv_bfloat16* grow = reinterpret_cast<__nv_bfloat16*>(prm.dQ) + it.b * prm.q_stride[0] +
                                  (long long)r * prm.q_stride[1] + it.hq * prm.q_stride[2] + half * DH;
            if (n_tiles == 0) {
                if (row_ok)
                    for (int e = 0; e < DH; e += 8) *reinterpret_cast<uint4*>(grow + e) = make_uint4(0, 0, 0, 0);
            } else {
                // dQ goes out through shared memory and one tiled TMA store per 64-column panel (a row-per-thread
                // store straight to global would touch 32 different lines per instruction).  The staging tile is
                // the dO buffer: every product that reads it has finished, and the producer may refill it only
                // after the arrival below.
                const float sc = prm.sm_scale;
                constexpr int kChunks = DH / 8;                       // 16-byte chunks this thread writes
                const int chunk0 = (half * DH % 64) / 8;              // first chunk inside the 128-byte panel row
                const uint32_t st_row = sDO + (uint32_t)((half * DH) / 64) * 16384 + (uint32_t)row * 128;
#pragma unroll
                for (int c = 0; c < DH / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_x32(tDq + lane_off + half * DH + c * 32, v);
                    tmem_wait_ld_dep(v);
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        const uint32_t x = pack_bf16(__uint_as_float(v[i]) * sc, __uint_as_float(v[i + 1]) * sc);
                        const uint32_t y = pack_bf16(__uint_as_float(v[i + 2]) * sc, __uint_as_float(v[i + 3]) * sc);
                        const uint32_t z = pack_bf16(__uint_as_float(v[i + 4]) * sc, __uint_as_float(v[i + 5]) * sc);
                        const uint32_t w = pack_bf16(__uint_as_float(v[i + 6]) * sc, __uint_as_float(v[i + 7]) * sc);
                        const int ch = chunk0 + c * 4 + i / 8;
                        st_shared_v4(st_row + (uint32_t)((ch ^ (row & 7)) << 4), x, y, z, w);
                    }
                }
                (void)kChunks;
                // the next item's first dQ product overwrites the accumulator; it is issued only after this
                // warp's next arrival on the dS barrier, which comes after the loads above
                tc_fence_before();
                fence_proxy_async_smem();
                ew_bar_sync();
                if (tid == kEwWarp0 * 32) {
                    for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                        tma_store_4d(&prm.tdq, sDO + pnl * 16384, pnl * 64, it.hq, r0, it.b);
                    bulk_commit_group();
                    bulk_wait_read_all();
                    mbar_arrive(bar(kBarDoEmpty));   // the dO buffer may take the next item's tile
                }
            }
            g += n_tiles;
        }
    }
    drain_if_failed();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem, 512);
    }
}

// ------------------------------------------------------------------------------------------
// dK/dV pass.  One CTA owns a 128-row key tile of one (batch, KV head) and loops over the query
// heads of the group and over the query tiles that read the key tile differentiably: the own
// segment from the diagonal on, plus the whole next segment when the tile reaches into the last
// T positions (the carried tail).  The loop set does not depend on the head flag.
// Transposed products keep the key on the accumulator row: S^T = K Q^T, dP^T = V dO^T,
// dV += P^T dO, dK += dS^T Q.  TMEM (512 columns): S^T at [0,128), dP^T at [128,256) (P^T and dS^T,
// bf16, are written over the start of each half of S^T and dP^T), dV at [256,256+D), dK at [384,384+D).
// Tensor-core order per (head, query tile) i:  dV(i) | S^T(i+1) | dK(i) | dP^T(i+1);  element-wise:
// B(i) runs during dV(i) and S^T(i+1), A(i+1) during dK(i) and dP^T(i+1).
template <int D>
struct DkvSmem {
    static constexpr int kPanels = D / 64;
    static constexpr uint32_t kTileBytes = kTile * D * 2;
    static constexpr int kStages = 2;
    static constexpr uint32_t kK = 0;
    static constexpr uint32_t kV = kTileBytes;
    static constexpr uint32_t kQ = 2 * kTileBytes;
    static constexpr uint32_t kDO = kQ + kStages * kTileBytes;
    static constexpr uint32_t kTotal = kDO + kStages * kTileBytes;
    static constexpr uint32_t kDynamic = kTotal + 1024;
};

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1) seg_attn_bwd_dkv_kernel(const __grid_constant__ BwdParams prm) {
    using SM = DkvSmem<D>;
    constexpr int trace_id = 2;
    (void)trace_id;
    TRACE_INIT();
    constexpr int NS = SM::kStages;
    enum { kBarKV = 0, kBarQFull = 1, kBarQEmpty = kBarQFull + NS, kBarDoFull = kBarQEmpty + NS,
           kBarDoEmpty = kBarDoFull + NS, kBarSFull = kBarDoEmpty + NS, kBarDpFull, kBarPFull, kBarDsFull, kBarDone,
           kNumBars };
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[kNumBars];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(16) float s_lse[2][kTile];
    __shared__ __align__(16) float s_dsum[2][kTile];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sKt = smem_base + SM::kK, sVt = smem_base + SM::kV;
    auto sQ = [&](int s) { return smem_base + SM::kQ + s * SM::kTileBytes; };
    auto sDO = [&](int s) { return smem_base + SM::kDO + s * SM::kTileBytes; };
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    // Work item: the grid is laid out as (KV head, batch) x (segment) x (rank of the tile inside its
    // segment).  Neighbouring CTAs thus read the same query tiles (L2 reuse), and inside a segment the
    // heavy tiles come first: the tiles of the carried tail (read by two segments), then the segment's
    // tiles from its first on (the earlier the tile, the more query tiles follow it), so that the grid
    // ends with short items.  Positions past the last key tile are empty.
    const int n_bs = prm.heads.n_slots * prm.B;
    const int rank = (int)(blockIdx.x % (unsigned)prm.dkv_tps);
    const int rem = (int)(blockIdx.x / (unsigned)prm.dkv_tps);
    const int seg = rem % prm.dkv_n_seg, bs = rem / prm.dkv_n_seg;
    (void)n_bs;
    const int k_in_seg = rank < prm.dkv_tail_tiles ? prm.dkv_tps - prm.dkv_tail_tiles + rank : rank - prm.dkv_tail_tiles;
    const int kt = seg * prm.dkv_tps + k_in_seg;
    if (kt >= prm.n_kvtiles) return;
    const int slot = bs % prm.heads.n_slots;
    const int b = bs / prm.heads.n_slots;
    const int hq0 = prm.heads.logical[slot] * prm.g;
    const MaskGeom& geo = prm.geom;
    const int c0 = kt * kTile;
    long long rq_lo, rq_hi;
    const int cls = prm.heads.flag[slot];
    kv_tile_q_range(geo, c0, cls, &rq_lo, &rq_hi);
    const int qt_lo = (int)(rq_lo / kTile);
    const int n_qt = rq_hi >= rq_lo ? (int)(rq_hi / kTile) - qt_lo + 1 : 0;
    const int n_it = n_qt * prm.g;

    if (tid == 0) {
        for (int i = 0; i < kNumBars; ++i)
            mbar_init(bar(i), (i == kBarPFull || i == kBarDsFull) ? kEwWarps : 1);
        fence_mbar_init();
        prefetch_tmap(&prm.tq);
        prefetch_tmap(&prm.tk);
        prefetch_tmap(&prm.tv);
        prefetch_tmap(&prm.tdo);
    }
    __syncwarp();
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const uint32_t tSt = tmem, tDpt = tmem + 128, tDv = tmem + 256, tDk = tmem + 384;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && n_it > 0) {
            mbar_expect_tx(bar(kBarKV), 2 * SM::kTileBytes);
            for (int pnl = 0; pnl < SM::kPanels; ++pnl) {
                tma_load_4d(sKt + pnl * 16384, &prm.tk, bar(kBarKV), pnl * 64, slot, c0, b);
                tma_load_4d(sVt + pnl * 16384, &prm.tv, bar(kBarKV), pnl * 64, slot, c0, b);
            }
            for (int i = 0; i < n_it; ++i) {
                const int s = i % NS, ph = (i / NS) & 1;
                const int hq = hq0 + i / n_qt;
                const int row = (qt_lo + i % n_qt) * kTile;
                if (!mbar_wait(bar(kBarQEmpty + s), ph ^ 1, 21)) break;
                mbar_expect_tx(bar(kBarQFull + s), SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                    tma_load_4d(sQ(s) + pnl * 16384, &prm.tq, bar(kBarQFull + s), pnl * 64, hq, row, b);
                if (!mbar_wait(bar(kBarDoEmpty + s), ph ^ 1, 27)) break;
                mbar_expect_tx(bar(kBarDoFull + s), SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                    tma_load_4d(sDO(s) + pnl * 16384, &prm.tdo, bar(kBarDoFull + s), pnl * 64, hq, row, b);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (whole warp, uniform control flow; one elected lane issues) ----------------
        if (n_it > 0) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t idesc_g = make_idesc_bf16(128, D, 0, 1);
            auto issue_st = [&](int i) -> bool {   // S^T(i) = K Q_i^T
                const int s = i % NS;
                if (!warp_wait(bar(kBarQFull + s), (i / NS) & 1, 23)) return false;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * 16384 + (k % 4) * 32;
                    mma_ss(tSt, make_sdesc(sKt + off, 16, 1024), make_sdesc(sQ(s) + off, 16, 1024), idesc_s, k > 0);
                }
                mma_commit(bar(kBarSFull));
                return true;
            };
            auto issue_dpt = [&](int i) -> bool {  // dP^T(i) = V dO_i^T
                const int s = i % NS;
                if (!warp_wait(bar(kBarDoFull + s), (i / NS) & 1, 28)) return false;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * 16384 + (k % 4) * 32;
                    mma_ss(tDpt, make_sdesc(sVt + off, 16, 1024), make_sdesc(sDO(s) + off, 16, 1024), idesc_s, k > 0);
                }
                mma_commit(bar(kBarDpFull));
                return true;
            };
            bool ok = warp_wait(bar(kBarKV), 0, 22);
            ok = ok && issue_st(0) && issue_dpt(0);
            for (int i = 0; ok && i < n_it; ++i) {
                const int s = i % NS;
                ok = warp_wait(bar(kBarPFull), i & 1, 24);
                if (!ok) break;
                tc_fence_after();
                TRACE(lane == 0, i * 8 + 4);
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k)
                    mma_ts(tDv, tSt + packed_a_col(k), make_sdesc(sDO(s) + k * 2048, 16384, 1024), idesc_g,
                           (i > 0) || (k > 0));
                mma_commit(bar(kBarDoEmpty + s));
                if (i + 1 < n_it) ok = issue_st(i + 1);
                if (!ok) break;
                TRACE(lane == 0, i * 8 + 5);
                ok = warp_wait(bar(kBarDsFull), i & 1, 29);
                if (!ok) break;
                tc_fence_after();
                TRACE(lane == 0, i * 8 + 6);
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k)
                    mma_ts(tDk, tDpt + packed_a_col(k), make_sdesc(sQ(s) + k * 2048, 16384, 1024), idesc_g,
                           (i > 0) || (k > 0));
                mma_commit(bar(kBarQEmpty + s));
                if (i + 1 < n_it) ok = issue_dpt(i + 1);
                TRACE(lane == 0, i * 8 + 7);
            }
            if (ok) mma_commit(bar(kBarDone));
        }
    } else if (warp >= kEwWarp0) {
        // ---------------- element-wise: thread = key row, 64 of the tile's 128 query columns ----------------
        const int quarter = warp & 3, half = (warp - kEwWarp0) >> 2;
        const int ctid = tid - kEwWarp0 * 32;      // 0..255 among the element-wise threads
        const int row = 32 * quarter + lane;       // key row of this thread inside the tile
        const uint32_t lane_off = (uint32_t)(32 * quarter) << 16;
        const uint32_t col_off = (uint32_t)half * 64;
        const int jl = c0 + row;
        const long long jpos = (long long)geo.kv_pos0 + jl;
        // query rows that read this key differentiably: [qlo, qhi]
        long long qlo_ll = jpos - geo.q_pos0, qhi_ll = hi_diff(geo, jpos < 0 ? 0 : jpos, cls) - 1 - geo.q_pos0;
        if (jpos < 0) qhi_ll = -1;
        if (qlo_ll < 0) qlo_ll = 0;
        if (qhi_ll > geo.Lq - 1) qhi_ll = geo.Lq - 1;
        const int qlo = (int)qlo_ll, qhi = (int)qhi_ll;
        // no element mask when every key row of the tile is read by every query row of the query tile
        const long long jfirst = (long long)geo.kv_pos0 + c0, jlast = jfirst + kTile - 1;
        const long long full_qlo = jlast - geo.q_pos0;  // latest first-reader
        long long full_qhi = (jfirst >= 0 ? hi_diff(geo, jfirst, cls) : 0) - 1 - geo.q_pos0;  // earliest last-reader
        if (full_qhi > geo.Lq - 1) full_qhi = geo.Lq - 1;
        const bool keys_in_range = c0 + kTile <= geo.kv_len && jfirst >= 0;

        const float sl2 = prm.scale_log2;
        // threads 0..127 stage LSE*log2e of the item's query rows, threads 128..255 the row dots D
        auto fetch_stat = [&](int i) -> float {
            const int hq = hq0 + i / n_qt;
            const int qr = (qt_lo + i % n_qt) * kTile + (ctid & 127);
            if (qr >= geo.Lq) return ctid < 128 ? INFINITY : 0.f;
            const long long si = ((long long)b * prm.Hq + hq) * geo.Lq + qr;
            if (ctid < 128) {
                const float l = prm.LSE[si];
                return (l == -INFINITY) ? INFINITY : l * kLog2e;
            }
            return prm.Dvec[si];
        };
        float stat_next = n_it > 0 ? fetch_stat(0) : 0.f;
        const uint64_t sl2x2 = f32x2(sl2, sl2);
        float P[64];
        // phase A: P^T = 2^(S^T*scale*log2e - LSE_q*log2e) (query = column), bf16 copy over the start of
        // this half of S^T
        auto phase_a = [&](auto masked_c, const int buf, const int q0) {
            constexpr bool MASKED = decltype(masked_c)::value;
            uint32_t sa_[32], sb_[32];
            tmem_ld_x32(tSt + lane_off + col_off, sa_);
            tmem_ld_x32(tSt + lane_off + col_off + 32, sb_);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t(&sv)[32] = c ? sb_ : sa_;
                tmem_wait_ld_dep(sv);
                uint32_t pk[16];
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const float4 l4 = *reinterpret_cast<const float4*>(&s_lse[buf][col_off + c * 32 + e]);
                    float t0, t1, t2, t3;
                    const uint64_t x01 = fma_f32x2(f32x2_bits(sv[e], sv[e + 1]), sl2x2, f32x2(-l4.x, -l4.y));
                    const uint64_t x23 = fma_f32x2(f32x2_bits(sv[e + 2], sv[e + 3]), sl2x2, f32x2(-l4.z, -l4.w));
                    float p0, p1, p2, p3;
                    f32x2_unpack(x01, t0, t1);
                    p0 = ex2(t0);
                    p1 = ex2(t1);
                    if (kDkvPolyEvery > 0 && (e / 4) % (kDkvPolyEvery > 0 ? kDkvPolyEvery : 1) == 0) {
                        ex2_poly_x2(x23, p2, p3);   // this pair on the FMA pipes: phase A is bound by the exp2 unit
                    } else {
                        f32x2_unpack(x23, t2, t3);
                        p2 = ex2(t2);
                        p3 = ex2(t3);
                    }
                    if (MASKED) {
                        const int q = q0 + (int)col_off + c * 32 + e;
                        p0 = (q >= qlo && q <= qhi) ? p0 : 0.f;
                        p1 = (q + 1 >= qlo && q + 1 <= qhi) ? p1 : 0.f;
                        p2 = (q + 2 >= qlo && q + 2 <= qhi) ? p2 : 0.f;
                        p3 = (q + 3 >= qlo && q + 3 <= qhi) ? p3 : 0.f;
                    }
                    P[c * 32 + e] = p0;
                    P[c * 32 + e + 1] = p1;
                    P[c * 32 + e + 2] = p2;
                    P[c * 32 + e + 3] = p3;
                    pk[e / 2] = pack_bf16(p0, p1);
                    pk[e / 2 + 1] = pack_bf16(p2, p3);
                }
                tmem_st_x16(tSt + lane_off + col_off + c * 16, pk);
            }
        };
        // phase B: dS^T = P^T * (dP^T - D_q), bf16, over the start of this half of dP^T
        auto phase_b = [&](const int buf) {
            uint32_t da_[32], db_[32];
            tmem_ld_x32(tDpt + lane_off + col_off, da_);
            tmem_ld_x32(tDpt + lane_off + col_off + 32, db_);
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t(&dv)[32] = c ? db_ : da_;
                tmem_wait_ld_dep(dv);
                uint32_t dk[16];
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const float4 d4 = *reinterpret_cast<const float4*>(&s_dsum[buf][col_off + c * 32 + e]);
                    float d0, d1, d2, d3;
                    f32x2_unpack(mul_f32x2(f32x2(P[c * 32 + e], P[c * 32 + e + 1]),
                                           add_f32x2(f32x2_bits(dv[e], dv[e + 1]), f32x2(-d4.x, -d4.y))), d0, d1);
                    f32x2_unpack(mul_f32x2(f32x2(P[c * 32 + e + 2], P[c * 32 + e + 3]),
                                           add_f32x2(f32x2_bits(dv[e + 2], dv[e + 3]), f32x2(-d4.z, -d4.w))), d2, d3);
                    dk[e / 2] = pack_bf16(d0, d1);
                    dk[e / 2 + 1] = pack_bf16(d2, d3);
                }
                tmem_st_x16(tDpt + lane_off + col_off + c * 16, dk);
            }
        };
        bool ok = true;
        for (int i = 0; i < n_it; ++i) {
            const int buf = i & 1;
            if (ctid < 128) s_lse[buf][ctid] = stat_next;
            else s_dsum[buf][ctid - 128] = stat_next;
            ew_bar_sync();
            if (i + 1 < n_it) stat_next = fetch_stat(i + 1);
            const int q0 = (qt_lo + i % n_qt) * kTile;
            const bool masked = !(keys_in_range && q0 >= full_qlo && q0 + kTile - 1 <= full_qhi);
            // after a failed wait keep looping (without touching TMEM) so that every element-wise thread
            // still reaches the named barrier above the same number of times
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull), i & 1, 25));
            if (!ok) continue;
            tc_fence_after();
            TRACE(tid == 128, i * 8 + 0);
            if (masked) phase_a(std::true_type{}, buf, q0);
            else phase_a(std::false_type{}, buf, q0);
            tmem_wait_st();
            ew_warp_arrive(bar(kBarPFull), lane);
            TRACE(tid == 128, i * 8 + 1);
            ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarDpFull), i & 1, 30));
            if (!ok) continue;
            tc_fence_after();
            TRACE(tid == 128, i * 8 + 2);
            phase_b(buf);
            tmem_wait_st();
            ew_warp_arrive(bar(kBarDsFull), lane);
            TRACE(tid == 128, i * 8 + 3);
        }
        if (n_it > 0 && ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarDone), 0, 26));
        tc_fence_after();
        constexpr int DH = D / 2;
        const bool row_ok = jl < geo.kv_len;
        __nv_bfloat16* gk = reinterpret_cast<__nv_bfloat16*>(prm.dK) + b * prm.k_stride[0] +
                            (long long)jl * prm.k_stride[1] + slot * prm.k_stride[2] + half * DH;
        __nv_bfloat16* gv = reinterpret_cast<__nv_bfloat16*>(prm.dV) + b * prm.v_stride[0] +
                            (long long)jl * prm.v_stride[1] + slot * prm.v_stride[2] + half * DH;
        if (n_it == 0) {
            if (row_ok)
                for (int e = 0; e < DH; e += 8) {
                    *reinterpret_cast<uint4*>(gk + e) = make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(gv + e) = make_uint4(0, 0, 0, 0);
                }
        } else if (ok) {
            // dV and dK go out through shared memory (the first dO and Q stages, idle by now) and tiled TMA
            // stores: a row-per-thread store straight to global would touch 32 different lines per instruction.
            // Rows past the end of the tensors are clipped by the stores.
            const float sc = prm.sm_scale;
            const int chunk0 = (half * DH % 64) / 8;  // first 16-byte chunk inside the 128-byte panel row
            const uint32_t row_off = (uint32_t)((half * DH) / 64) * 16384 + (uint32_t)row * 128;
#pragma unroll
            for (int c = 0; c < DH / 32; ++c) {
                uint32_t v[32], k[32];
                tmem_ld_x32(tDv + lane_off + half * DH + c * 32, v);
                tmem_ld_x32(tDk + lane_off + half * DH + c * 32, k);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; e += 8) {
                    const uint32_t sw = (uint32_t)(((chunk0 + c * 4 + e / 8) ^ (row & 7)) << 4);
                    st_shared_v4(sDO(0) + row_off + sw, pack_bf16(__uint_as_float(v[e]), __uint_as_float(v[e + 1])),
                                 pack_bf16(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3])),
                                 pack_bf16(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5])),
                                 pack_bf16(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7])));
                    st_shared_v4(sQ(0) + row_off + sw, pack_bf16(__uint_as_float(k[e]) * sc, __uint_as_float(k[e + 1]) * sc),
                                 pack_bf16(__uint_as_float(k[e + 2]) * sc, __uint_as_float(k[e + 3]) * sc),
                                 pack_bf16(__uint_as_float(k[e + 4]) * sc, __uint_as_float(k[e + 5]) * sc),
                                 pack_bf16(__uint_as_float(k[e + 6]) * sc, __uint_as_float(k[e + 7]) * sc));
                }
            }
            fence_proxy_async_smem();
        }
        // every element-wise thread reaches this barrier (also after a failed wait or with nothing to do)
        ew_bar_sync();
        if (tid == kEwWarp0 * 32 && n_it > 0 && ok) {
            for (int pnl = 0; pnl < SM::kPanels; ++pnl) {
                tma_store_4d(&prm.tdv, sDO(0) + pnl * 16384, pnl * 64, slot, c0, b);
                tma_store_4d(&prm.tdk, sQ(0) + pnl * 16384, pnl * 64, slot, c0, b);
            }
            bulk_commit_group();
            bulk_wait_all();
        }
    }
    drain_if_failed();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace segattn

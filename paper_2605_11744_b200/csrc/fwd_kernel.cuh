// Forward kernel: O = softmax(Q K^T * scale + mask) V and LSE (Appendix C, Eqs. "attn" and "ctx"),
// visiting only the key tiles the segment / tail / past-access mask leaves visible.
//
// Persistent: one CTA per SM walks a static list of work items (one 128-row query tile of one
// (batch, query head) each), heaviest items first, dealt round-robin to the CTAs.
// Roles (384 threads): warp 0 = TMA producer, warp 1 = tcgen05 issuer of the PV products and TMEM
// owner, warp 2 = tcgen05 issuer of the score products, warp 3 = scheduling warp (decodes the CTA's
// work items once and hands them to every other role through a ring in shared memory),
// warps 4..7 and 8..11 = two softmax groups (thread = query row) that take the key tiles of even
// and odd index in turn and pass the running row maximum on through shared memory, then share the
// epilogue.  The issuing warpgroup gives most of its registers to the softmax groups,
// whose threads hold a whole row of scores (128 values) in registers.
// TMEM (512 columns): one S buffer per softmax group at [0,256), one P buffer (bf16) per group at
// [256,384), O at [384,384+D).  A group reads its tile's scores out of TMEM once and hands the S
// buffer back at once, so the scores of its next tile are computed while it works on this one, and
// no product waits for another through a shared buffer: S(j+2) follows the read of S(j), PV(j)
// follows P(j).
#pragma once
#include <type_traits>

#include "mask.cuh"
#include "ptx.cuh"

namespace segattn {

constexpr int kFwdThreads = 384;
constexpr int kFwdEwWarp0 = 4;   // first softmax warp
constexpr int kFwdEwWarps = 8;
constexpr float kRescaleThreshold = 8.0f;  // lazy O rescale: only when the row max grows by > 2^8
constexpr int kFwdPolyChains = 0;     // of every four pairs of scores, this many take 2^x from the FMA pipes (ex2_poly_x2)
constexpr int kFwdExpTurnChunk = 2;   // a group hands the exp2 unit on after this 32-column chunk (of 0..3) of its tile
constexpr int kFwdRing = 8;           // decoded work items in flight between the scheduling warp and the other roles
constexpr int kFwdDescReaders = 12;   // readers of a decoded item: producer (twice: Q cursor and K/V cursor), two issuers, eight softmax warps
constexpr int kFwdRegsIssue = 56;     // registers per thread of warps 0..3 after the re-partitioning
constexpr int kFwdRegsSoftmax = 224;  // and of the softmax warps (128 * 80 + 256 * 208 <= 384 * 168)

template <int D>
struct FwdSmem {
    static constexpr int kPanels = D / 64;               // 64-column (128-byte) panels per tile
    static constexpr uint32_t kTileBytes = kTile * D * 2;  // one 128-row tile of Q, K or V
    static constexpr int kQStages = 1, kKStages = 2, kVStages = 2;
    static constexpr uint32_t kQ = 0;
    static constexpr uint32_t kK = kQStages * kTileBytes;
    static constexpr uint32_t kV = kK + kKStages * kTileBytes;
    static constexpr uint32_t kOut = kV + kVStages * kTileBytes;  // staging tile of O for the tiled store
    static constexpr uint32_t kTotal = kOut + kTileBytes;
#ifdef SEGATTN_TRACE
    static constexpr uint32_t kTraceSlots = 3072;  // debug builds: clock stamps are kept in shared memory until the end
#else
    static constexpr uint32_t kTraceSlots = 0;
#endif
    static constexpr uint32_t kDynamic = kTotal + 1024 + kTraceSlots * 8;  // 1024: slack to align the base to 1024 B
};

#ifdef SEGATTN_TRACE
// In this kernel a stamp goes to shared memory (a global store per stamp would sit in front of the
// kernel's own fences and distort what is measured); the traced CTA copies the stamps out at the end.
#undef TRACE
#define TRACE(cond, idx) do { if (trace_on_ && (cond) && (uint32_t)(idx) < SM::kTraceSlots) { long long t_; asm volatile("mov.u64 %0, %clock64;" : "=l"(t_)); asm volatile("st.shared.b64 [%0], %1;" :: "r"(smem_trace + (uint32_t)(idx) * 8u), "l"(t_)); } } while (0)
#endif

// A decoded work item as the scheduling warp publishes it in shared memory (32 bytes): the item and
// its visible key tiles [t_lo, t_lo + n).  n = 0: nothing visible (the rows are written as zeros);
// n < 0: end of this CTA's list.
struct FwdDesc {
    int b, hq, slot, qt, cls, t_lo, n;
};
using FwdItem = WorkItem;
__device__ __forceinline__ FwdItem fwd_decode(const FwdParams& prm, int idx) { return decode_item(prm, idx); }
// first visible key tile and number of visible key tiles of a work item
__device__ __forceinline__ void fwd_item_tiles(const FwdParams& prm, const FwdItem& it, int* t_lo, int* n_tiles) {
    long long jl_lo, jl_hi;
    q_tile_kv_range<true>(prm.geom, it.qt * kTile, it.cls, false, &jl_lo, &jl_hi);
    *t_lo = (int)(jl_lo / kTile);
    *n_tiles = jl_hi >= jl_lo ? (int)(jl_hi / kTile) - *t_lo + 1 : 0;
}

// Hand-over of the running row maximum from the softmax group that finished the maximum pass of
// tile j to the group that works on tile j + 1: named barrier 2 + (j & 1), 128 threads arrive
// (without waiting) and 128 wait.
__device__ __forceinline__ void fwd_m_arrive(int parity) { asm volatile("bar.arrive %0, 256;" ::"r"(2 + parity) : "memory"); }
__device__ __forceinline__ void fwd_m_sync(int parity) { asm volatile("bar.sync %0, 256;" ::"r"(2 + parity) : "memory"); }
// barrier of all eight softmax warps
__device__ __forceinline__ void fwd_groups_sync() { asm volatile("bar.sync 4, 256;" ::: "memory"); }

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1) seg_attn_fwd_kernel(const __grid_constant__ FwdParams prm) {
    using SM = FwdSmem<D>;
    constexpr int trace_id = 0;
    (void)trace_id;
    TRACE_INIT();
    constexpr int NQ = SM::kQStages, NK = SM::kKStages, NV = SM::kVStages;
    enum { kBarQFull = 0, kBarQEmpty = kBarQFull + NQ, kBarKFull = kBarQEmpty + NQ, kBarKEmpty = kBarKFull + NK,
           kBarVFull = kBarKEmpty + NK, kBarVEmpty = kBarVFull + NV, kBarSFull = kBarVEmpty + NV, kBarSFree = kBarSFull + 2,
           kBarPFull = kBarSFree + 2, kBarExp = kBarPFull + 2, kBarPvDone = kBarExp + 8, kBarOFull = kBarPvDone + 2, kBarDescFull = kBarOFull + 1,
           kBarDescEmpty = kBarDescFull + kFwdRing, kNumBars = kBarDescEmpty + kFwdRing };
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[kNumBars];
    __shared__ uint32_t tmem_slot;
    __shared__ float s_m[2][kTile];       // [tile parity][row]: running row maximum after that tile
    __shared__ float s_fin[2][3][kTile];  // [group][m, l, c][row]: the groups' partial sums, once per work item
    __shared__ __align__(16) int s_desc[kFwdRing][8];  // ring of decoded work items (FwdDesc)

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    auto sQ = [&](int s) { return smem_base + SM::kQ + s * SM::kTileBytes; };
    auto sK = [&](int s) { return smem_base + SM::kK + s * SM::kTileBytes; };
    auto sV = [&](int s) { return smem_base + SM::kV + s * SM::kTileBytes; };
    const uint32_t sOut = smem_base + SM::kOut;
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    const MaskGeom& geo = prm.geom;
#ifdef SEGATTN_TRACE
    const uint32_t smem_trace = smem_base + SM::kTotal;
    if (trace_on_)
        for (uint32_t i = tid; i < SM::kTraceSlots; i += kFwdThreads)
            asm volatile("st.shared.b64 [%0], %1;" ::"r"(smem_trace + i * 8u), "l"(0ll));
#endif

    if (tid == 0) {
        prefetch_tmap(&prm.to);
        for (int i = 0; i < kNumBars; ++i)
            mbar_init(bar(i), (i >= kBarSFree && i < kBarExp) ? kFwdEwWarps / 2  // S-free, P-full: one arrival per warp
                              : i >= kBarDescEmpty                ? kFwdDescReaders
                                                                  : 1);
        fence_mbar_init();
        prefetch_tmap(&prm.tq);
        prefetch_tmap(&prm.tk);
        prefetch_tmap(&prm.tv);
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
    const uint32_t tS0 = tmem, tP0 = tmem + 256, tO = tmem + 384;  // S and P buffers of group g at tS0 + 128 g, tP0 + 64 g
    // The k-th work item of this CTA as the scheduling warp decoded it (called by a whole warp or by one
    // lane of it; `leader` marks the one thread that hands the ring slot back).  False: a wait gave up.
    auto read_desc = [&](int k, FwdDesc* d, bool whole_warp, bool leader) -> bool {
        const int rs = k % kFwdRing;
        if (!mbar_wait<true>(bar(kBarDescFull + rs), (uint32_t)(k / kFwdRing) & 1, 14)) return false;
        const uint32_t a = smem_u32(&s_desc[rs][0]);
        int pad;
        ld_shared_v4(a, d->b, d->hq, d->slot, d->qt);
        ld_shared_v4(a + 16, d->cls, d->t_lo, d->n, pad);
        if (whole_warp) __syncwarp();
        if (leader) mbar_arrive(bar(kBarDescEmpty + rs));
        return true;
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        setmaxnreg_dec<kFwdRegsIssue>();
        if (lane == 0) {
            int kq = 0;           // Q cursor: runs ahead, the next item whose Q is not requested yet
            bool q_more = true;   // the Q cursor has not reached the end of the list
            int qn_ld = 0;        // Q tiles requested so far
            bool ok = true;
            // request the Q tile of the next work item that has visible key tiles, if there is one
            auto advance_q = [&]() {
                while (ok && q_more) {
                    FwdDesc it;
                    if (!(ok = read_desc(kq++, &it, false, true))) return;
                    if (it.n < 0) {
                        q_more = false;
                        return;
                    }
                    if (it.n == 0) continue;
                    const int qs = qn_ld % NQ;
                    if (!(ok = mbar_wait<true>(bar(kBarQEmpty + qs), ((qn_ld / NQ) & 1) ^ 1, 1))) return;
                    mbar_expect_tx(bar(kBarQFull + qs), SM::kTileBytes);
                    for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                        tma_load_4d(sQ(qs) + pnl * 16384, &prm.tq, bar(kBarQFull + qs), pnl * 64, it.hq, it.qt * kTile, it.b);
                    ++qn_ld;
                    return;
                }
            };
            int g = 0;  // key tiles requested so far (all work items; far fewer than 2^31)
            advance_q();
            for (int kd = 0; ok; ++kd) {
                FwdDesc it;
                if (!(ok = read_desc(kd, &it, false, true)) || it.n < 0) break;
                const int t_lo = it.t_lo, n = it.n;
                if (n == 0) continue;
                auto load_k = [&](int j) -> bool {
                    const int gj = g + j;
                    const int s = (int)(gj % NK);
                    if (!mbar_wait<true>(bar(kBarKEmpty + s), (uint32_t)((gj / NK) & 1) ^ 1, 2)) return false;
                    mbar_expect_tx(bar(kBarKFull + s), SM::kTileBytes);
                    for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                        tma_load_4d(sK(s) + pnl * 16384, &prm.tk, bar(kBarKFull + s), pnl * 64, it.slot, (t_lo + n - 1 - j) * kTile,
                                    it.b);
                    return true;
                };
                auto load_v = [&](int j) -> bool {
                    const int gj = g + j;
                    const int s = (int)(gj % NV);
                    if (!mbar_wait<true>(bar(kBarVEmpty + s), (uint32_t)((gj / NV) & 1) ^ 1, 3)) return false;
                    mbar_expect_tx(bar(kBarVFull + s), SM::kTileBytes);
                    for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                        tma_load_4d(sV(s) + pnl * 16384, &prm.tv, bar(kBarVFull + s), pnl * 64, it.slot, (t_lo + n - 1 - j) * kTile,
                                    it.b);
                    return true;
                };
                // K runs two tiles ahead of V, as the scores do of the PV products
                ok = ok && load_k(0);
                if (ok && n > 1) ok = load_k(1);
                for (int j = 0; ok && j < n; ++j) {
                    if (j + 2 < n) ok = load_k(j + 2);
                    if (ok) ok = load_v(j);
                }
                g += n;
                advance_q();  // the next item's Q: its buffer is free once this item's last scores are issued
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer for O += P V (whole warp, uniform control flow; one elected lane issues) -------
        // The two kinds of product are issued by two warps on different schedulers, so that neither
        // waits behind the other's barriers and each has half the issue work.
        setmaxnreg_dec<kFwdRegsIssue>();
        constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);
        static_assert(NV == 2 && NK == 2 && NQ == 1, "ring indices below are written out for these depths");
        int g = 0;  // key tiles of earlier work items (a CTA sees far fewer than 2^31)
        bool ok = true;
        // What the two issuers execute between a barrier and their first product is kept short: everything
        // that does not depend on the barrier is worked out before the wait, the waits of one batch share
        // one vote, and optional completion signals are predicated.
        for (int kd = 0; ok; ++kd) {
            FwdDesc it;
            ok = __all_sync(0xffffffffu, read_desc(kd, &it, true, lane == 0));
            if (!ok || it.n < 0) break;
            const int n = it.n;
            if (n == 0) continue;
            for (int j = 0; j < n; ++j) {
                const int gj = g + j;
                const int sv = gj & 1;
                const uint32_t ph = (uint32_t)(gj >> 1) & 1;
                const uint32_t a_p = tP0 + (uint32_t)sv * 64;
                const uint64_t vd = make_sdesc(sV(sv), 16384, 1024);
                // V tile landed, P written (the two barriers share ring position and phase)
                if (!(ok = warp_wait2<true>(bar(kBarVFull + sv), ph, bar(kBarPFull + sv), ph, 6))) break;
                tc_fence_after();
                TRACE(lane == 0, j * 16 + 4);
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k)
                    mma_ts(tO, a_p + k * 8, vd + ((k * 2048) >> 4), idesc_pv, (j > 0) || (k > 0));
                mma_commit(bar(kBarPvDone + sv));  // P(j) is consumed and O holds tile j
                mma_commit(bar(kBarVEmpty + sv));
                mma_commit_if(j == n - 1, bar(kBarOFull));  // the item's O is complete
                TRACE(lane == 0, j * 16 + 5);
            }
            g += n;
        }
    } else if (warp == 2) {
        // ---------------- MMA issuer for S = Q K^T (whole warp; one elected lane issues) ----------------
        setmaxnreg_dec<kFwdRegsIssue>();
        constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, 0, 0);
        int qn = 0;  // work items with visible tiles started so far
        int g = 0;   // key tiles of earlier work items
        bool ok = true;
        const uint64_t qd = make_sdesc(sQ(0), 16, 1024);
        for (int kd = 0; ok; ++kd) {
            FwdDesc it;
            ok = __all_sync(0xffffffffu, read_desc(kd, &it, true, lane == 0));
            if (!ok || it.n < 0) break;
            const int n = it.n;
            if (n == 0) continue;
            if (!(ok = warp_wait<true>(bar(kBarQFull), (uint32_t)qn & 1, 4))) break;
            ++qn;
            for (int j = 0; j < n; ++j) {
                const int gj = g + j;
                const int s = gj & 1;  // softmax group of the tile = its S buffer = its place in the K ring
                const uint32_t d_s = tS0 + (uint32_t)s * 128;
                const uint64_t kd = make_sdesc(sK(s), 16, 1024);
                // The group has read the scores of tile gj - 2 out of this buffer (the first two tiles of a
                // launch find fresh buffers: parity 1 of a new barrier reads complete); and the K tile has landed.
                const uint32_t ph = (uint32_t)(gj >> 1) & 1;
                if (!(ok = warp_wait2<true>(bar(kBarSFree + s), ph ^ 1, bar(kBarKFull + s), ph, 12))) break;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = ((k / 4) * 16384 + (k % 4) * 32) >> 4;  // descriptor addresses count 16-byte units
                    mma_ss(d_s, qd + off, kd + off, idesc_qk, k > 0);
                }
                mma_commit(bar(kBarSFull + s));  // first: a softmax group waits for it
                mma_commit(bar(kBarKEmpty + s));
                mma_commit_if(j == n - 1, bar(kBarQEmpty));  // the item's last scores release Q
                TRACE(lane == 0, j * 16 + 6);
            }
            g += n;
        }
    } else if (warp < kFwdEwWarp0) {
        // ---------------- scheduling warp: decodes this CTA's work items once, for every other role ----------------
        setmaxnreg_dec<kFwdRegsIssue>();
        if (lane == 0) {
            ItemWalk walk(blockIdx.x, gridDim.x, prm.n_items);
            bool more = true;
            for (int k = 0; more; ++k) {
                const int rs = k % kFwdRing;
                // every reader has taken the item that was in this slot (a fresh barrier reads complete for parity 1)
                if (!mbar_wait<true>(bar(kBarDescEmpty + rs), ((uint32_t)(k / kFwdRing) & 1) ^ 1, 15)) break;
                int item, t_lo = 0, n = -1;
                FwdItem it = {0, 0, 0, 0, 0};
                if ((more = walk.next(&item))) {
                    it = fwd_decode(prm, item);
                    fwd_item_tiles(prm, it, &t_lo, &n);
                }
                const uint32_t a = smem_u32(&s_desc[rs][0]);
                st_shared_v4(a, (uint32_t)it.b, (uint32_t)it.hq, (uint32_t)it.slot, (uint32_t)it.qt);
                st_shared_v4(a + 16, (uint32_t)it.cls, (uint32_t)t_lo, (uint32_t)n, 0u);
                mbar_arrive(bar(kBarDescFull + rs));  // release: the stores above are visible to whoever sees the arrival
            }
        }
    } else {
        // ---------------- softmax + epilogue ----------------
        setmaxnreg_inc<kFwdRegsSoftmax>();
        // Two groups of four warps; thread = query row (all 128 key columns of a tile).  Group 0 takes the
        // key tiles of even global index, group 1 the odd ones, so that one group's maximum pass and
        // hand-offs run under the other group's exponentials.  The running maximum travels from tile to
        // tile through shared memory; each group keeps its own partial row sum.
        const int quarter = warp & 3, grp = (warp - kFwdEwWarp0) >> 2;
        const int row = 32 * quarter + lane;
        const uint32_t lane_off = (uint32_t)(32 * quarter) << 16;
        constexpr int DH = D / 2;  // this group's share of an O row in the epilogue
        const float sl2 = prm.scale_log2;
        const uint64_t sl2x2 = f32x2(sl2, sl2);
        int g = 0;   // key tiles of earlier work items (a CTA sees far fewer than 2^31)
        int qn = 0;  // earlier work items that had visible tiles
        bool ok = true;
        for (int kd = 0; ok; ++kd) {
            FwdDesc it;
            ok = __all_sync(0xffffffffu, read_desc(kd, &it, true, lane == 0));
            if (!ok || it.n < 0) break;
            const int t_lo = it.t_lo, n_tiles = it.n;
            const int r0 = it.qt * kTile;
            const int r = r0 + row;
            const long long p = (long long)geo.q_pos0 + r;
            // visible local key rows of this query row: [vlo, vhi]
            long long vlo_ll = lo_visible<true>(geo, p, it.cls) - geo.kv_pos0;
            long long vhi_ll = p - geo.kv_pos0;
            if (vlo_ll < 0) vlo_ll = 0;
            if (vhi_ll > geo.kv_len - 1) vhi_ll = geo.kv_len - 1;
            const int vlo = (int)vlo_ll, vhi = (int)vhi_ll;
            // a key tile [c0, c0+128) needs no element mask when every row of the tile sees all of it
            long long full_lo = lo_visible<true>(geo, (long long)geo.q_pos0 + r0 + kTile - 1, it.cls) - geo.kv_pos0;
            long long full_hi = (long long)geo.q_pos0 + r0 - geo.kv_pos0;
            if (full_hi > geo.kv_len - 1) full_hi = geo.kv_len - 1;

            // m_used: the running maximum this group's sums are scaled by.  l_run: sum of the unrounded p of
            // this group's tiles (gives LSE).  c_run: sum over those tiles of (bf16(p) - p) for the tile's
            // largest p.  O is divided by l + c, i.e. by a row sum in which the dominant probability
            // enters as the bf16 value the PV product really used, so that a row where one key dominates
            // (outlier keys) stays a convex combination of value rows.
            float m_used = -INFINITY, l_run = 0.f, c_run = 0.f;
            TRACE(tid == 128, 2048 + qn * 4 + 0);
            // One key tile of the online softmax.  One copy of the code serves masked and fully visible tiles
            // (the mask is applied to the scores in registers, under a branch): the kernel's instruction
            // footprint, not the branch, is what costs time here.
            auto softmax_tile = [&](const bool MASKED, const int j, const int gj, const int c0) {
                const uint32_t tSj = tS0 + (uint32_t)grp * 128 + lane_off;
                const uint32_t tPj = tP0 + (uint32_t)grp * 64 + lane_off;
                // the whole row of scores into registers, then the S buffer goes back to the issuer
                uint32_t sc[4][32];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld_x32(tSj + c * 32, sc[c]);
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_wait_ld_dep(sc[c]);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarSFree + grp));
                if (MASKED) {
                    // visible columns of this row inside the tile: [lo_t, hi_t] (tile-local, compared with constants)
                    const int lo_t = vlo - c0, hi_t = vhi - c0;
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int i = 0; i < 32; ++i) mask_score(sc[c][i], lo_t, hi_t, c * 32 + i);
                }
                // row maximum of the raw scores
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        mx0 = fmax3(mx0, __uint_as_float(sc[c][i]), __uint_as_float(sc[c][i + 1]));
                        mx1 = fmax3(mx1, __uint_as_float(sc[c][i + 2]), __uint_as_float(sc[c][i + 3]));
                        mx2 = fmax3(mx2, __uint_as_float(sc[c][i + 4]), __uint_as_float(sc[c][i + 5]));
                        mx3 = fmax3(mx3, __uint_as_float(sc[c][i + 6]), __uint_as_float(sc[c][i + 7]));
                    }
                // the pairs of maximum chain k are the pairs (i / 2) % 4 == k; the last kFwdPolyChains chains are the
                // pairs whose exponentials come from the polynomial
                const float mx_unit = kFwdPolyChains >= 2 ? fmaxf(mx0, mx1) : kFwdPolyChains == 1 ? fmax3(mx0, mx1, mx2)
                                                                                                : fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                const float mx_poly = kFwdPolyChains >= 2 ? fmaxf(mx2, mx3) : kFwdPolyChains == 1 ? mx3 : -INFINITY;
                const float mx = fmaxf(mx_unit, mx_poly);
                // running maximum after the previous tile (the other group's), then this tile's
                float m_prev = -INFINITY;
                if (j > 0) {
                    fwd_m_sync((int)((gj - 1) & 1));
                    m_prev = s_m[(gj - 1) & 1][row];
                }
                TRACE((tid & 127) == 0, j * 16 + 1);
                const float m_tile = mx * sl2;  // scale > 0, so the maximum commutes with the scaling
                const bool grow = m_tile > m_prev + kRescaleThreshold || (m_prev == -INFINITY && m_tile > -INFINITY);
                const float m_new = grow ? m_tile : m_prev;
                if (j + 1 < n_tiles) {
                    s_m[gj & 1][row] = m_new;
                    __threadfence_block();
                    fwd_m_arrive((int)(gj & 1));
                }
                TRACE((tid & 127) == 0, j * 16 + 12);
                if (m_new > m_used) {  // bring this group's sums to the current scale
                    const float f = ex2(m_used - m_new);  // 0 when nothing was accumulated yet
                    l_run *= f;
                    c_run *= f;
                    m_used = m_new;
                }
                if (j > 0 && __any_sync(0xffffffffu, grow)) {
                    // PV(j-1), which accumulates into O, may still be running: wait for it
                    ok = __all_sync(0xffffffffu,
                                    mbar_wait<true>(bar(kBarPvDone + (int)((gj - 1) & 1)), (uint32_t)(((gj - 1) >> 1) & 1), 10));
                    if (!ok) return;
                    tc_fence_after();
                    const float alpha = grow ? ex2(m_prev - m_new) : 1.f;
#pragma unroll 1  // rare (the row maximum has grown by more than the threshold): kept small, not fast
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t v[32];
                        tmem_ld_x32(tO + lane_off + c * 32, v);
                        tmem_wait_ld_dep(v);
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                        tmem_st_x32(tO + lane_off + c * 32, v);
                    }
                }
                TRACE((tid & 127) == 0, j * 16 + 13);
                // this group's P buffer is free: PV(j-2) has read it (long since true as a rule)
                if (gj >= 2) {
                    ok = __all_sync(0xffffffffu,
                                    mbar_wait<true>(bar(kBarPvDone + (int)(gj & 1)), (uint32_t)(((gj - 2) >> 1) & 1), 11));
                    if (!ok) return;
                }
                TRACE((tid & 127) == 0, j * 16 + 14);
                // The two warps of a scheduler (one of each group) take turns at the exponentials: they share
                // the scheduler's exp2 unit.  This pass starts when the other warp's pass over tile gj - 1 is
                // nearly through, so that one group's loads, maximum and hand-overs run under the other's
                // exponentials instead of beside them.
                if (kFwdExpTurnChunk >= 0 && gj >= 1) {
                    ok = __all_sync(0xffffffffu, mbar_wait<true>(bar(kBarExp + (int)((gj - 1) & 1) * 4 + quarter),
                                                                 (uint32_t)(((gj - 1) >> 1) & 1), 13));
                    if (!ok) return;
                }
                TRACE((tid & 127) == 0, j * 16 + 7);
                // p = 2^(s*scale*log2e - m); row sum from the unrounded p; P to TMEM as bf16
                const float m_eff = (m_new == -INFINITY) ? 0.f : m_new;
                const uint64_t nm2 = f32x2(-m_eff, -m_eff);
                {
                    // the tile's largest p, exactly as formed below (by the exp2 unit or by the polynomial)
                    const float tm = fmaf(mx, sl2, -m_eff);
                    float pm = ex2(tm);
                    if (kFwdPolyChains > 0 && mx_poly > mx_unit) {
                        float q0, q1;
                        ex2_poly_x2(f32x2(tm, tm), q0, q1);
                        pm = q0;
                    }
                    const uint32_t pr = pack_bf16(pm, 0.f);
                    c_run += __uint_as_float(pr << 16) - pm;
                }
                uint64_t acc_a = 0ull, acc_b = 0ull;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const uint64_t t = fma_f32x2(f32x2_bits(sc[c][i], sc[c][i + 1]), sl2x2, nm2);
                        float p0, p1;
                        if ((i / 2) % 4 >= 4 - kFwdPolyChains) {
                            ex2_poly_x2(t, p0, p1);
                        } else {
                            float t0, t1;
                            f32x2_unpack(t, t0, t1);
                            p0 = ex2(t0);
                            p1 = ex2(t1);
                        }
                        if (i & 2) acc_b = add_f32x2(acc_b, f32x2(p0, p1));
                        else acc_a = add_f32x2(acc_a, f32x2(p0, p1));
                        pk[i / 2] = pack_bf16(p0, p1);
                    }
                    tmem_st_x16(tPj + c * 16, pk);
                    TRACE((tid & 127) == 0, j * 16 + 8 + c);
                    if (c == kFwdExpTurnChunk) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kBarExp + grp * 4 + quarter));
                        if (c < 3) reg_fence32(sc[c < 3 ? c + 1 : 3]);  // the rest of the pass stays behind the hand-over
                    }
                }
                {
                    float s0, s1;
                    f32x2_unpack(add_f32x2(acc_a, acc_b), s0, s1);
                    l_run += s0 + s1;
                }
            };
            for (int j = 0; j < n_tiles; ++j) {
                const int gj = g + j;
                if ((gj & 1) != grp) continue;  // the other group's tile
                const int c0 = (t_lo + n_tiles - 1 - j) * kTile;
                const bool masked = !(c0 >= full_lo && c0 + kTile - 1 <= full_hi);
                TRACE((tid & 127) == 0, j * 16 + 3);
                ok = __all_sync(0xffffffffu, mbar_wait<true>(bar(kBarSFull + grp), (uint32_t)((gj >> 1) & 1), 8));
                if (!ok) break;
                tc_fence_after();
                TRACE((tid & 127) == 0, j * 16 + 0);
                softmax_tile(masked, j, gj, c0);
                if (!ok) break;
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPFull + grp));
                TRACE((tid & 127) == 0, j * 16 + 2);
            }
            if (!ok) break;
            TRACE(tid == 128, 2048 + qn * 4 + 1);
            // ---------------- epilogue of the work item ----------------
            float m_fin = -INFINITY, l_tot = 0.f, lc_tot = 0.f;
            if (n_tiles > 0) {
                // the previous item's O tile has left the staging buffer
                if (tid == kFwdEwWarp0 * 32) bulk_wait_read_all();
                // the groups combine their partial sums at the final scale
                s_fin[grp][0][row] = m_used;
                s_fin[grp][1][row] = l_run;
                s_fin[grp][2][row] = c_run;
                fwd_groups_sync();
                const float m_o = s_fin[grp ^ 1][0][row], l_o = s_fin[grp ^ 1][1][row], c_o = s_fin[grp ^ 1][2][row];
                m_fin = fmaxf(m_used, m_o);
                const float f_me = (m_used == -INFINITY) ? 0.f : ex2(m_used - m_fin);
                const float f_o = (m_o == -INFINITY) ? 0.f : ex2(m_o - m_fin);
                // same order of additions in both groups, so that they divide by the same number
                const float l_g0 = grp == 0 ? l_run * f_me : l_o * f_o, l_g1 = grp == 0 ? l_o * f_o : l_run * f_me;
                const float c_g0 = grp == 0 ? c_run * f_me : c_o * f_o, c_g1 = grp == 0 ? c_o * f_o : c_run * f_me;
                l_tot = l_g0 + l_g1;
                lc_tot = l_tot + (c_g0 + c_g1);
                // one completion per work item: every PV product of the item has finished
                ok = __all_sync(0xffffffffu, mbar_wait<true>(bar(kBarOFull), (uint32_t)(qn & 1), 9));
                if (!ok) break;
                tc_fence_after();
                TRACE(tid == 128, 2048 + qn * 4 + 2);
                ++qn;
            }
            const bool have = n_tiles > 0 && l_tot > 0.f && lc_tot > 0.f;
            const float inv_l = have ? 1.f / lc_tot : 0.f;
            if (r < geo.Lq && grp == 0)
                prm.LSE[((long long)it.b * prm.Hq + it.hq) * geo.Lq + r] =
                    have ? (m_fin + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
            if (n_tiles == 0) {
                __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(prm.O) + it.b * prm.o_stride[0] +
                                      (long long)r * prm.o_stride[1] + it.hq * prm.o_stride[2] + grp * DH;
                if (r < geo.Lq)
                    for (int e = 0; e < DH; e += 8) *reinterpret_cast<uint4*>(orow + e) = make_uint4(0, 0, 0, 0);
            } else {
                // O goes out through shared memory and one tiled TMA store per 64-column panel (a row-per-thread
                // store straight to global would touch 32 different lines per instruction); rows past the end
                // of the tensor are clipped by the store
                const int chunk0 = (grp * DH % 64) / 8;  // first 16-byte chunk inside the 128-byte panel row
                const uint32_t st_row = sOut + (uint32_t)((grp * DH) / 64) * 16384 + (uint32_t)row * 128;
#pragma unroll
                for (int c = 0; c < DH / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_x32(tO + lane_off + grp * DH + c * 32, v);
                    tmem_wait_ld_dep(v);
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        const uint32_t x = pack_bf16(__uint_as_float(v[i]) * inv_l, __uint_as_float(v[i + 1]) * inv_l);
                        const uint32_t y = pack_bf16(__uint_as_float(v[i + 2]) * inv_l, __uint_as_float(v[i + 3]) * inv_l);
                        const uint32_t z = pack_bf16(__uint_as_float(v[i + 4]) * inv_l, __uint_as_float(v[i + 5]) * inv_l);
                        const uint32_t w = pack_bf16(__uint_as_float(v[i + 6]) * inv_l, __uint_as_float(v[i + 7]) * inv_l);
                        const int ch = chunk0 + c * 4 + i / 8;
                        st_shared_v4(st_row + (uint32_t)((ch ^ (row & 7)) << 4), x, y, z, w);
                    }
                }
                // Both groups have read O and the exchanged sums before either starts the next item: its
                // first PV product (which overwrites O) needs a P arrival that comes after this barrier.
                tc_fence_before();
                fence_proxy_async_smem();
                fwd_groups_sync();
                if (tid == kFwdEwWarp0 * 32) {
                    for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                        tma_store_4d(&prm.to, sOut + pnl * 16384, pnl * 64, it.hq, r0, it.b);
                    bulk_commit_group();
                }
                TRACE(tid == 128, 2048 + (qn - 1) * 4 + 3);
            }
            g += n_tiles;
        }
    }
    // ---------------- teardown ----------------
    if (tid == kFwdEwWarp0 * 32) bulk_wait_all();  // the last O tile has been written
    drain_if_failed();
    tc_fence_before();
    __syncthreads();
#ifdef SEGATTN_TRACE
    if (trace_on_)
        for (uint32_t i = tid; i < SM::kTraceSlots; i += kFwdThreads) {
            long long t_;
            asm volatile("ld.shared.b64 %0, [%1];" : "=l"(t_) : "r"(smem_trace + i * 8u));
            g_trace[i] = t_;
        }
#endif
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace segattn

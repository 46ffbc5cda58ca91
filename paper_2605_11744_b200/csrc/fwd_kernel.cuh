// Forward kernel: O = softmax(Q K^T * scale + mask) V and LSE for one 128-row query tile of one
// (batch, query head) per CTA (Appendix C, Eqs. "attn" and "ctx"), visiting only the key tiles
// the segment / tail / past-access mask leaves visible.
//
// Roles (192 threads): warp 0 = TMA producer, warp 1 = tcgen05 MMA issuer and TMEM owner,
// warps 2..5 = softmax + epilogue (thread <-> query row through the 32x32b TMEM shape).
// TMEM (256 columns): S / P at columns [0,128) (P, bf16, aliases the first 64), O at [128,128+D).
// Two CTAs are resident per SM so that one CTA's softmax overlaps the other's MMAs.
#pragma once
#include <type_traits>

#include "mask.cuh"
#include "ptx.cuh"

namespace segattn {

constexpr int kFwdThreads = 192;
constexpr float kRescaleThreshold = 8.0f;  // lazy O rescale: only when the row max grows by > 2^8

template <int D>
struct FwdSmem {
    static constexpr int kPanels = D / 64;               // 64-column (128-byte) panels per tile
    static constexpr uint32_t kTileBytes = kTile * D * 2;  // one 128-row tile of Q, K or V
    static constexpr uint32_t kQ = 0;
    static constexpr uint32_t kK = kTileBytes;
    static constexpr uint32_t kV = 2 * kTileBytes;
    static constexpr uint32_t kTotal = 3 * kTileBytes;
    static constexpr uint32_t kDynamic = kTotal + 1024;  // slack to align the base to 1024 B
};

enum FwdBar { kBarQ = 0, kBarKFull, kBarKEmpty, kBarVFull, kBarVEmpty, kBarSFull, kBarPFull, kBarOFull, kFwdBars };

// Decode blockIdx.x into a work item, heaviest first: flagged heads (long visible ranges)
// before the others, late query tiles before early ones.
struct FwdItem {
    int b, hq, slot, qt;
    bool flagged;
};
__device__ __forceinline__ FwdItem fwd_decode(const FwdParams& prm, int idx) {
    const HeadTable& ht = prm.heads;
    const int per_f = ht.n_flagged * prm.g * prm.B;
    const int per_u = (ht.n_slots - ht.n_flagged) * prm.g * prm.B;
    const int n_f = per_f * prm.n_qtiles;
    FwdItem it;
    int hb, cls_off, cls_n;
    if (idx < n_f) {
        it.qt = prm.n_qtiles - 1 - idx / per_f;
        hb = idx % per_f;
        cls_off = 0;
        cls_n = ht.n_flagged;
    } else {
        idx -= n_f;
        it.qt = prm.n_qtiles - 1 - idx / per_u;
        hb = idx % per_u;
        cls_off = ht.n_flagged;
        cls_n = ht.n_slots - ht.n_flagged;
    }
    const int r = hb % prm.g;
    const int t = hb / prm.g;
    it.slot = ht.order[cls_off + t % cls_n];
    it.b = t / cls_n;
    it.hq = ht.logical[it.slot] * prm.g + r;
    it.flagged = ht.flag[it.slot] != 0;
    return it;
}

template <int D>
__global__ void __launch_bounds__(kFwdThreads, 2) seg_attn_fwd_kernel(const __grid_constant__ FwdParams prm) {
    using SM = FwdSmem<D>;
    constexpr int trace_id = 0;
    (void)trace_id;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[kFwdBars];
    __shared__ uint32_t tmem_slot;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + SM::kQ, sK = smem_base + SM::kK, sV = smem_base + SM::kV;
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    const FwdItem it = fwd_decode(prm, blockIdx.x);
    const MaskGeom& geo = prm.geom;
    const int r0 = it.qt * kTile;
    long long jl_lo, jl_hi;
    q_tile_kv_range(geo, r0, it.flagged, false, &jl_lo, &jl_hi);
    const int t_lo = (int)(jl_lo / kTile);
    const int n_tiles = jl_hi >= jl_lo ? (int)(jl_hi / kTile) - t_lo + 1 : 0;

    if (tid == 0) {
        mbar_init(bar(kBarQ), 1);
        mbar_init(bar(kBarKFull), 1);
        mbar_init(bar(kBarKEmpty), 1);
        mbar_init(bar(kBarVFull), 1);
        mbar_init(bar(kBarVEmpty), 1);
        mbar_init(bar(kBarSFull), 1);
        mbar_init(bar(kBarPFull), 128);
        mbar_init(bar(kBarOFull), 1);
        fence_mbar_init();
        prefetch_tmap(&prm.tq);
        prefetch_tmap(&prm.tk);
        prefetch_tmap(&prm.tv);
    }
    __syncwarp();
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const uint32_t tS = tmem, tP = tmem, tO = tmem + 128;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && n_tiles > 0) {
            mbar_expect_tx(bar(kBarQ), SM::kTileBytes);
            for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                tma_load_4d(sQ + pnl * 16384, &prm.tq, bar(kBarQ), pnl * 64, it.hq, r0, it.b);
            for (int j = 0; j < n_tiles; ++j) {
                const int row = (t_lo + j) * kTile;
                if (!mbar_wait(bar(kBarKEmpty), (j & 1) ^ 1, 1)) break;
                mbar_expect_tx(bar(kBarKFull), SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                    tma_load_4d(sK + pnl * 16384, &prm.tk, bar(kBarKFull), pnl * 64, it.slot, row, it.b);
                if (!mbar_wait(bar(kBarVEmpty), (j & 1) ^ 1, 2)) break;
                mbar_expect_tx(bar(kBarVFull), SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                    tma_load_4d(sV + pnl * 16384, &prm.tv, bar(kBarVFull), pnl * 64, it.slot, row, it.b);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (whole warp, uniform control flow; one elected lane issues) ----------------
        if (n_tiles > 0) {
            constexpr uint32_t idesc_qk = make_idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 0, 1);
            auto issue_qk = [&]() {
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * 16384 + (k % 4) * 32;
                    mma_ss(tS, make_sdesc(sQ + off, 16, 1024), make_sdesc(sK + off, 16, 1024), idesc_qk, k > 0);
                }
            };
            bool ok = warp_wait(bar(kBarQ), 0, 3) && warp_wait(bar(kBarKFull), 0, 4);
            if (ok) {
                tc_fence_after();
                issue_qk();
                mma_commit(bar(kBarKEmpty));
                mma_commit(bar(kBarSFull));
            }
            for (int j = 0; ok && j < n_tiles; ++j) {
                ok = warp_wait(bar(kBarPFull), j & 1, 5) && warp_wait(bar(kBarVFull), j & 1, 6);
                if (!ok) break;
                tc_fence_after();
                TRACE(lane == 0, j * 8 + 4);
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k)
                    mma_ts(tO, tP + k * 8, make_sdesc(sV + k * 2048, 16384, 1024), idesc_pv, (j > 0) || (k > 0));
                mma_commit(bar(kBarVEmpty));
                TRACE(lane == 0, j * 8 + 5);
                if (j + 1 < n_tiles) {
                    ok = warp_wait(bar(kBarKFull), (j + 1) & 1, 7);
                    if (!ok) break;
                    tc_fence_after();
                    TRACE(lane == 0, j * 8 + 6);
                    issue_qk();
                    TRACE(lane == 0, j * 8 + 7);
                    mma_commit(bar(kBarKEmpty));
                    mma_commit(bar(kBarSFull));
                } else {
                    mma_commit(bar(kBarOFull));
                }
            }
        }
    } else {
        // ---------------- softmax + epilogue: one thread per query row ----------------
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_off = (uint32_t)(32 * (warp & 3)) << 16;
        const int r = r0 + row;
        const long long p = (long long)geo.q_pos0 + r;
        // visible local key rows of this query row: [vlo, vhi]
        long long vlo_ll = lo_visible(geo, p, it.flagged) - geo.kv_pos0;
        long long vhi_ll = p - geo.kv_pos0;
        if (vlo_ll < 0) vlo_ll = 0;
        if (vhi_ll > geo.kv_len - 1) vhi_ll = geo.kv_len - 1;
        const int vlo = (int)vlo_ll, vhi = (int)vhi_ll;
        // a key tile [c0, c0+128) needs no element mask when every row of the tile sees all of it
        long long full_lo = lo_visible(geo, (long long)geo.q_pos0 + r0 + kTile - 1, it.flagged) - geo.kv_pos0;
        long long full_hi = (long long)geo.q_pos0 + r0 - geo.kv_pos0;
        if (full_hi > geo.kv_len - 1) full_hi = geo.kv_len - 1;

        const float sl2 = prm.scale_log2;
        const uint64_t sl2x2 = f32x2(sl2, sl2);
        // l_run: row sum of the unrounded p (gives LSE).  c_run: sum over tiles of (bf16(p) - p) for the
        // tile's largest p.  O is divided by l_run + c_run, i.e. by a row sum in which the dominant
        // probability enters as the bf16 value the PV product really used, so that a row where one key
        // dominates (outlier keys) stays a convex combination of value rows.
        float m_run = -INFINITY, l_run = 0.f, c_run = 0.f;
        bool ok = true;
        // One key tile of the online softmax.  MASKED is a compile-time flag so that the common,
        // fully visible tile runs straight-line code (no per-element tests, no branches that would keep
        // the scheduler from overlapping the exp latency of neighbouring elements).
        auto softmax_tile = [&](auto masked_c, const int j, const int c0) {
            constexpr bool MASKED = decltype(masked_c)::value;
            uint32_t va[32], vb[32];
            // pass 1: row maximum of the raw scores; the load of chunk c+1 is in flight while chunk c is reduced
            float mx0 = -INFINITY, mx1 = -INFINITY;
            tmem_ld_x32(tS + lane_off, va);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t(&cur)[32] = (c & 1) ? vb : va;
                uint32_t(&nxt)[32] = (c & 1) ? va : vb;
                tmem_wait_ld_dep(cur);
                tmem_ld_x32(tS + lane_off + ((c + 1) & 3) * 32, nxt);  // c == 3: chunk 0 again, for pass 2
                if (MASKED) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int col = c0 + c * 32 + i;
                        cur[i] = (col >= vlo && col <= vhi) ? cur[i] : 0xff800000u;  // -inf
                    }
                }
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    mx0 = fmax3(mx0, __uint_as_float(cur[i]), __uint_as_float(cur[i + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(cur[i + 2]), __uint_as_float(cur[i + 3]));
                }
            }
            const float mx = fmaxf(mx0, mx1);
            TRACE(tid == 64, j * 8 + 1);
            const float m_tile = mx * sl2;  // scale > 0, so the maximum commutes with the scaling
            const float m_new = fmaxf(m_run, m_tile);
            const bool grow = m_new > m_run + kRescaleThreshold || (m_run == -INFINITY && m_new > -INFINITY);
            float alpha = 1.f;
            if (grow) {
                alpha = ex2(m_run - m_new);  // 0 when nothing was accumulated yet
                l_run *= alpha;
                c_run *= alpha;
                m_run = m_new;
            }
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
                // every MMA issued before this tile's S (the previous PV included) has retired
                tmem_wait_ld_dep(va);  // the prefetched chunk 0: drain before reusing the load path
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_x32(tO + lane_off + c * 32, v);
                    tmem_wait_ld_dep(v);
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                    tmem_st_x32(tO + lane_off + c * 32, v);
                }
            }
            // pass 2: p = 2^(s*scale*log2e - m); row sum from the unrounded p; P to TMEM as bf16
            const float m_eff = (m_run == -INFINITY) ? 0.f : m_run;
            const uint64_t nm2 = f32x2(-m_eff, -m_eff);
            {
                const float pm = ex2(fmaf(mx, sl2, -m_eff));  // the tile's largest p, exactly as pass 2 forms it
                const uint32_t pr = pack_bf16(pm, 0.f);
                c_run += __uint_as_float(pr << 16) - pm;
            }
            uint64_t acc_a = 0ull, acc_b = 0ull;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t(&cur)[32] = (c & 1) ? vb : va;
                uint32_t(&nxt)[32] = (c & 1) ? va : vb;
                tmem_wait_ld_dep(cur);
                if (c < 3) tmem_ld_x32(tS + lane_off + (c + 1) * 32, nxt);
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const uint64_t t = fma_f32x2(f32x2_bits(cur[i], cur[i + 1]), sl2x2, nm2);
                    float t0, t1;
                    f32x2_unpack(t, t0, t1);
                    float p0 = ex2(t0), p1 = ex2(t1);
                    if (MASKED) {
                        const int col = c0 + c * 32 + i;
                        p0 = (col >= vlo && col <= vhi) ? p0 : 0.f;
                        p1 = (col + 1 >= vlo && col + 1 <= vhi) ? p1 : 0.f;
                    }
                    if (i & 2) acc_b = add_f32x2(acc_b, f32x2(p0, p1));
                    else acc_a = add_f32x2(acc_a, f32x2(p0, p1));
                    pk[i / 2] = pack_bf16(p0, p1);
                }
                tmem_st_x16(tP + lane_off + c * 16, pk);
            }
            {
                float s0, s1;
                f32x2_unpack(add_f32x2(acc_a, acc_b), s0, s1);
                l_run += s0 + s1;
            }
        };
        for (int j = 0; j < n_tiles; ++j) {
            const int c0 = (t_lo + j) * kTile;
            const bool masked = !(c0 >= full_lo && c0 + kTile - 1 <= full_hi);
            ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull), j & 1, 8));
            if (!ok) break;
            tc_fence_after();
            TRACE(tid == 64, j * 8 + 0);
            if (masked) softmax_tile(std::true_type{}, j, c0);
            else softmax_tile(std::false_type{}, j, c0);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(kBarPFull));
            TRACE(tid == 64, j * 8 + 2);
        }
        // ---------------- epilogue ----------------
        if (n_tiles > 0 && ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarOFull), 0, 9));
        tc_fence_after();
        const bool have = n_tiles > 0 && ok && l_run > 0.f && l_run + c_run > 0.f;
        const float inv_l = have ? 1.f / (l_run + c_run) : 0.f;
        if (r < geo.Lq && (ok || n_tiles == 0)) {
            __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(prm.O) + it.b * prm.o_stride[0] +
                                  (long long)r * prm.o_stride[1] + it.hq * prm.o_stride[2];
            prm.LSE[((long long)it.b * prm.Hq + it.hq) * geo.Lq + r] =
                have ? (m_run + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
            if (!have) {
                for (int e = 0; e < D; e += 8) *reinterpret_cast<uint4*>(orow + e) = make_uint4(0, 0, 0, 0);
            }
        }
        if (n_tiles > 0 && ok) {
            __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(prm.O) + it.b * prm.o_stride[0] +
                                  (long long)r * prm.o_stride[1] + it.hq * prm.o_stride[2];
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t v[32];
                tmem_ld_x32(tO + lane_off + c * 32, v);
                tmem_wait_ld_dep(v);
                if (r < geo.Lq && have) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(v[i]) * inv_l, __uint_as_float(v[i + 1]) * inv_l);
                        o.y = pack_bf16(__uint_as_float(v[i + 2]) * inv_l, __uint_as_float(v[i + 3]) * inv_l);
                        o.z = pack_bf16(__uint_as_float(v[i + 4]) * inv_l, __uint_as_float(v[i + 5]) * inv_l);
                        o.w = pack_bf16(__uint_as_float(v[i + 6]) * inv_l, __uint_as_float(v[i + 7]) * inv_l);
                        *reinterpret_cast<uint4*>(orow + c * 32 + i) = o;
                    }
                }
            }
        }
    }
    // ---------------- teardown ----------------
    drain_if_failed();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem, 256);
    }
}

}  // namespace segattn

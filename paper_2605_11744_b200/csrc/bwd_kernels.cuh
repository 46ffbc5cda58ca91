// Backward kernels (softmax VJP with the stop-gradient rule of Definition 3.2 / Lemma B.1):
//   bwd_rowdot_kernel   D_p = <dO_p, O_p>                                    (HBM-bound)
//   seg_attn_bwd_dq_kernel    dQ_p = scale * sum_{visible j} dS_pj K_j             (sg keys included)
//   seg_attn_bwd_dkv_kernel   dK_j = scale * sum_{diff(p,j)} dS_pj Q_p,  dV_j = sum_{diff(p,j)} P_pj dO_p
// with P = 2^(s*scale*log2e - LSE*log2e), dS = P * (dO V^T - D).  Both tensor-core kernels use
// the role split of the forward kernel: warp 0 TMA producer, warp 1 tcgen05 issuer and TMEM
// owner, warps 2..5 element-wise work with one thread per accumulator row.  No atomics: a CTA
// owns its output tile, so results are bitwise reproducible.
#pragma once
#include <type_traits>

#include "mask.cuh"
#include "ptx.cuh"

namespace segattn {

constexpr int kBwdThreads = 192;
constexpr float kLog2e = 1.4426950408889634f;

// ------------------------------------------------------------------------------------------
// D[b][h][r] = sum_e dO[b][r][h][e] * O[b][r][h][e]; one group of D/8 threads per row, 16-byte loads.
template <int D>
__global__ void __launch_bounds__(256) bwd_rowdot_kernel(const __nv_bfloat16* __restrict__ O,
                                                         const __nv_bfloat16* __restrict__ dO, float* __restrict__ Dvec,
                                                         int B, int Lq, int Hq, long long s0, long long s1,
                                                         long long s2) {
    constexpr int TPR = D / 8;  // threads per row
    const long long n_rows = (long long)B * Lq * Hq;
    const long long row = (long long)blockIdx.x * (256 / TPR) + threadIdx.x / TPR;
    const int part = threadIdx.x % TPR;
    float acc = 0.f;
    int b = 0, r = 0, h = 0;
    if (row < n_rows) {
        h = (int)(row % Hq);
        r = (int)((row / Hq) % Lq);
        b = (int)(row / ((long long)Hq * Lq));
        const long long off = b * s0 + (long long)r * s1 + h * s2 + part * 8;
        const uint4 a = *reinterpret_cast<const uint4*>(O + off);
        const uint4 g = *reinterpret_cast<const uint4*>(dO + off);
        const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
        const __nv_bfloat162* pg = reinterpret_cast<const __nv_bfloat162*>(&g);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 x = __bfloat1622float2(pa[i]), y = __bfloat1622float2(pg[i]);
            acc = fmaf(x.x, y.x, acc);
            acc = fmaf(x.y, y.y, acc);
        }
    }
#pragma unroll
    for (int o = TPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (row < n_rows && part == 0) Dvec[((long long)b * Hq + h) * Lq + r] = acc;
}

// ------------------------------------------------------------------------------------------
// dQ pass.  TMEM (512 columns): S / dS at [0,128) (dS, bf16, aliases the first 64),
// dP at [128,256), dQ accumulator at [256,256+D).
template <int D>
struct DqSmem {
    static constexpr int kPanels = D / 64;
    static constexpr uint32_t kTileBytes = kTile * D * 2;
    static constexpr int kStages = 2;
    static constexpr uint32_t kQ = 0;
    static constexpr uint32_t kDO = kTileBytes;
    static constexpr uint32_t kK = 2 * kTileBytes;
    static constexpr uint32_t kV = kK + kStages * kTileBytes;
    static constexpr uint32_t kTotal = kV + kStages * kTileBytes;
    static constexpr uint32_t kDynamic = kTotal + 1024;
};

struct DqItem {
    int b, hq, slot, qt;
    bool flagged;
};
__device__ __forceinline__ DqItem dq_decode(const BwdParams& prm, int idx) {
    const HeadTable& ht = prm.heads;
    const int per_f = ht.n_flagged * prm.g * prm.B;
    const int per_u = (ht.n_slots - ht.n_flagged) * prm.g * prm.B;
    const int n_f = per_f * prm.n_qtiles;
    DqItem it;
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
__global__ void __launch_bounds__(kBwdThreads, 1) seg_attn_bwd_dq_kernel(const __grid_constant__ BwdParams prm) {
    using SM = DqSmem<D>;
    constexpr int NS = SM::kStages;
    enum { kBarQ = 0, kBarKFull = 1, kBarKEmpty = 1 + NS, kBarVFull = 1 + 2 * NS, kBarVEmpty = 1 + 3 * NS,
           kBarSFull = 1 + 4 * NS, kBarDsFull, kBarDqFull, kNumBars };
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[kNumBars];
    __shared__ uint32_t tmem_slot;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + SM::kQ, sDO = smem_base + SM::kDO;
    auto sK = [&](int s) { return smem_base + SM::kK + s * SM::kTileBytes; };
    auto sV = [&](int s) { return smem_base + SM::kV + s * SM::kTileBytes; };
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    const DqItem it = dq_decode(prm, blockIdx.x);
    const MaskGeom& geo = prm.geom;
    const int r0 = it.qt * kTile;
    long long jl_lo, jl_hi;
    q_tile_kv_range(geo, r0, it.flagged, false, &jl_lo, &jl_hi);
    const int t_lo = (int)(jl_lo / kTile);
    const int n_tiles = jl_hi >= jl_lo ? (int)(jl_hi / kTile) - t_lo + 1 : 0;

    if (tid == 0) {
        for (int i = 0; i < kNumBars; ++i) mbar_init(bar(i), i == kBarDsFull ? 128 : 1);
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
    const uint32_t tS = tmem, tDs = tmem, tDp = tmem + 128, tDq = tmem + 256;

    if (warp == 0) {
        if (lane == 0 && n_tiles > 0) {
            mbar_expect_tx(bar(kBarQ), 2 * SM::kTileBytes);
            for (int pnl = 0; pnl < SM::kPanels; ++pnl) {
                tma_load_4d(sQ + pnl * 16384, &prm.tq, bar(kBarQ), pnl * 64, it.hq, r0, it.b);
                tma_load_4d(sDO + pnl * 16384, &prm.tdo, bar(kBarQ), pnl * 64, it.hq, r0, it.b);
            }
            for (int j = 0; j < n_tiles; ++j) {
                const int s = j % NS, ph = (j / NS) & 1;
                const int row = (t_lo + j) * kTile;
                if (!mbar_wait(bar(kBarKEmpty + s), ph ^ 1, 11)) break;
                mbar_expect_tx(bar(kBarKFull + s), SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                    tma_load_4d(sK(s) + pnl * 16384, &prm.tk, bar(kBarKFull + s), pnl * 64, it.slot, row, it.b);
                if (!mbar_wait(bar(kBarVEmpty + s), ph ^ 1, 12)) break;
                mbar_expect_tx(bar(kBarVFull + s), SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl)
                    tma_load_4d(sV(s) + pnl * 16384, &prm.tv, bar(kBarVFull + s), pnl * 64, it.slot, row, it.b);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && n_tiles > 0) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, 0, 1);
            bool ok = mbar_wait(bar(kBarQ), 0, 13);
            for (int j = 0; ok && j < n_tiles; ++j) {
                const int s = j % NS, ph = (j / NS) & 1;
                ok = mbar_wait(bar(kBarKFull + s), ph, 14) && mbar_wait(bar(kBarVFull + s), ph, 15);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * 16384 + (k % 4) * 32;
                    mma_ss(tS, make_sdesc(sQ + off, 16, 1024), make_sdesc(sK(s) + off, 16, 1024), idesc_s, k > 0);
                }
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * 16384 + (k % 4) * 32;
                    mma_ss(tDp, make_sdesc(sDO + off, 16, 1024), make_sdesc(sV(s) + off, 16, 1024), idesc_s, k > 0);
                }
                mma_commit(bar(kBarVEmpty + s));
                mma_commit(bar(kBarSFull));
                ok = mbar_wait(bar(kBarDsFull), j & 1, 16);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k)
                    mma_ts(tDq, tDs + k * 8, make_sdesc(sK(s) + k * 2048, 16384, 1024), idesc_dq, (j > 0) || (k > 0));
                mma_commit(bar(kBarKEmpty + s));
            }
            if (ok) mma_commit(bar(kBarDqFull));
        }
    } else {
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_off = (uint32_t)(32 * (warp & 3)) << 16;
        const int r = r0 + row;
        const long long p = (long long)geo.q_pos0 + r;
        long long vlo_ll = lo_visible(geo, p, it.flagged) - geo.kv_pos0;
        long long vhi_ll = p - geo.kv_pos0;
        if (vlo_ll < 0) vlo_ll = 0;
        if (vhi_ll > geo.kv_len - 1) vhi_ll = geo.kv_len - 1;
        const int vlo = (int)vlo_ll, vhi = (int)vhi_ll;
        long long full_lo = lo_visible(geo, (long long)geo.q_pos0 + r0 + kTile - 1, it.flagged) - geo.kv_pos0;
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
        const float sl2 = prm.scale_log2;
        const uint64_t sl2x2 = f32x2(sl2, sl2);
        const uint64_t nlse2 = f32x2(-lse2, -lse2);
        const uint64_t ndsum2 = f32x2(-dsum, -dsum);
        // dS = P * (dP - D) for one key tile; MASKED is a compile-time flag so that fully visible
        // tiles run branch-free straight-line code
        auto ds_tile = [&](auto masked_c, const int c0) {
            constexpr bool MASKED = decltype(masked_c)::value;
            uint32_t sa_[32], sb_[32], da_[32], db_[32];
            tmem_ld_x32(tS + lane_off, sa_);
            tmem_ld_x32(tDp + lane_off, da_);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t(&sv)[32] = (c & 1) ? sb_ : sa_;
                uint32_t(&dv)[32] = (c & 1) ? db_ : da_;
                uint32_t(&sn)[32] = (c & 1) ? sa_ : sb_;
                uint32_t(&dn)[32] = (c & 1) ? da_ : db_;
                tmem_wait_ld_dep(sv);
                tmem_wait_ld_dep(dv);
                if (c < 3) {
                    tmem_ld_x32(tS + lane_off + (c + 1) * 32, sn);
                    tmem_ld_x32(tDp + lane_off + (c + 1) * 32, dn);
                }
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float t0, t1;
                    f32x2_unpack(fma_f32x2(f32x2_bits(sv[i], sv[i + 1]), sl2x2, nlse2), t0, t1);
                    const uint64_t p2 = f32x2(ex2(t0), ex2(t1));
                    const uint64_t ds2 = mul_f32x2(p2, add_f32x2(f32x2_bits(dv[i], dv[i + 1]), ndsum2));
                    float d0, d1;
                    f32x2_unpack(ds2, d0, d1);
                    if (MASKED) {
                        const int col = c0 + c * 32 + i;
                        d0 = (col >= vlo && col <= vhi) ? d0 : 0.f;
                        d1 = (col + 1 >= vlo && col + 1 <= vhi) ? d1 : 0.f;
                    }
                    pk[i / 2] = pack_bf16(d0, d1);
                }
                tmem_st_x16(tDs + lane_off + c * 16, pk);
            }
        };
        bool ok = true;
        for (int j = 0; j < n_tiles; ++j) {
            const int c0 = (t_lo + j) * kTile;
            const bool masked = !(c0 >= full_lo && c0 + kTile - 1 <= full_hi);
            ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull), j & 1, 17));
            if (!ok) break;
            tc_fence_after();
            if (masked) ds_tile(std::true_type{}, c0);
            else ds_tile(std::false_type{}, c0);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(kBarDsFull));
        }
        if (n_tiles > 0 && ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarDqFull), 0, 18));
        tc_fence_after();
        __nv_bfloat16* grow = reinterpret_cast<__nv_bfloat16*>(prm.dQ) + it.b * prm.q_stride[0] +
                              (long long)r * prm.q_stride[1] + it.hq * prm.q_stride[2];
        if (n_tiles == 0) {
            if (row_ok)
                for (int e = 0; e < D; e += 8) *reinterpret_cast<uint4*>(grow + e) = make_uint4(0, 0, 0, 0);
        } else if (ok) {
            const float sc = prm.sm_scale;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t v[32];
                tmem_ld_x32(tDq + lane_off + c * 32, v);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(v[i]) * sc, __uint_as_float(v[i + 1]) * sc);
                        o.y = pack_bf16(__uint_as_float(v[i + 2]) * sc, __uint_as_float(v[i + 3]) * sc);
                        o.z = pack_bf16(__uint_as_float(v[i + 4]) * sc, __uint_as_float(v[i + 5]) * sc);
                        o.w = pack_bf16(__uint_as_float(v[i + 6]) * sc, __uint_as_float(v[i + 7]) * sc);
                        *reinterpret_cast<uint4*>(grow + c * 32 + i) = o;
                    }
                }
            }
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
// dV += P^T dO, dK += dS^T Q.  TMEM (512 columns): S^T / P^T at [0,128), dP^T / dS^T at [128,256)
// (the bf16 forms alias the first 64 columns of each), dV at [256,256+D), dK at [384,384+D).
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

__device__ __forceinline__ void compute_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1) seg_attn_bwd_dkv_kernel(const __grid_constant__ BwdParams prm) {
    using SM = DkvSmem<D>;
    constexpr int NS = SM::kStages;
    enum { kBarKV = 0, kBarQFull = 1, kBarQEmpty = 1 + NS, kBarSFull = 1 + 2 * NS, kBarPFull, kBarDone, kNumBars };
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

    // work item: key tiles in reverse order (late tiles first), then KV head, then batch
    const int kt = prm.n_kvtiles - 1 - (int)(blockIdx.x % prm.n_kvtiles);
    const int slot = (int)((blockIdx.x / prm.n_kvtiles) % prm.heads.n_slots);
    const int b = (int)(blockIdx.x / ((long long)prm.n_kvtiles * prm.heads.n_slots));
    const int hq0 = prm.heads.logical[slot] * prm.g;
    const MaskGeom& geo = prm.geom;
    const int c0 = kt * kTile;
    long long rq_lo, rq_hi;
    kv_tile_q_range(geo, c0, &rq_lo, &rq_hi);
    const int qt_lo = (int)(rq_lo / kTile);
    const int n_qt = rq_hi >= rq_lo ? (int)(rq_hi / kTile) - qt_lo + 1 : 0;
    const int n_it = n_qt * prm.g;

    if (tid == 0) {
        for (int i = 0; i < kNumBars; ++i) mbar_init(bar(i), i == kBarPFull ? 128 : 1);
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
    const uint32_t tSt = tmem, tPt = tmem, tDpt = tmem + 128, tDst = tmem + 128, tDv = tmem + 256, tDk = tmem + 384;

    if (warp == 0) {
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
                mbar_expect_tx(bar(kBarQFull + s), 2 * SM::kTileBytes);
                for (int pnl = 0; pnl < SM::kPanels; ++pnl) {
                    tma_load_4d(sQ(s) + pnl * 16384, &prm.tq, bar(kBarQFull + s), pnl * 64, hq, row, b);
                    tma_load_4d(sDO(s) + pnl * 16384, &prm.tdo, bar(kBarQFull + s), pnl * 64, hq, row, b);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && n_it > 0) {
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t idesc_g = make_idesc_bf16(128, D, 0, 1);
            bool ok = mbar_wait(bar(kBarKV), 0, 22);
            for (int i = 0; ok && i < n_it; ++i) {
                const int s = i % NS, ph = (i / NS) & 1;
                ok = mbar_wait(bar(kBarQFull + s), ph, 23);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * 16384 + (k % 4) * 32;
                    mma_ss(tSt, make_sdesc(sKt + off, 16, 1024), make_sdesc(sQ(s) + off, 16, 1024), idesc_s, k > 0);
                }
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * 16384 + (k % 4) * 32;
                    mma_ss(tDpt, make_sdesc(sVt + off, 16, 1024), make_sdesc(sDO(s) + off, 16, 1024), idesc_s, k > 0);
                }
                mma_commit(bar(kBarSFull));
                ok = mbar_wait(bar(kBarPFull), i & 1, 24);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k)
                    mma_ts(tDv, tPt + k * 8, make_sdesc(sDO(s) + k * 2048, 16384, 1024), idesc_g, (i > 0) || (k > 0));
#pragma unroll
                for (int k = 0; k < kTile / 16; ++k)
                    mma_ts(tDk, tDst + k * 8, make_sdesc(sQ(s) + k * 2048, 16384, 1024), idesc_g, (i > 0) || (k > 0));
                mma_commit(bar(kBarQEmpty + s));
            }
            if (ok) mma_commit(bar(kBarDone));
        }
    } else {
        const int ctid = tid - 64;  // 0..127 among the compute warps
        const int row = 32 * (warp & 3) + lane;  // key row of this thread inside the tile
        const uint32_t lane_off = (uint32_t)(32 * (warp & 3)) << 16;
        const int jl = c0 + row;
        const long long jpos = (long long)geo.kv_pos0 + jl;
        // query rows that read this key differentiably: [qlo, qhi]
        long long qlo_ll = jpos - geo.q_pos0, qhi_ll = hi_diff(geo, jpos < 0 ? 0 : jpos) - 1 - geo.q_pos0;
        if (jpos < 0) qhi_ll = -1;
        if (qlo_ll < 0) qlo_ll = 0;
        if (qhi_ll > geo.Lq - 1) qhi_ll = geo.Lq - 1;
        const int qlo = (int)qlo_ll, qhi = (int)qhi_ll;
        // no element mask when every key row of the tile is read by every query row of the query tile
        const long long jfirst = (long long)geo.kv_pos0 + c0, jlast = jfirst + kTile - 1;
        const long long full_qlo = jlast - geo.q_pos0;  // latest first-reader
        long long full_qhi = (jfirst >= 0 ? hi_diff(geo, jfirst) : 0) - 1 - geo.q_pos0;  // earliest last-reader
        if (full_qhi > geo.Lq - 1) full_qhi = geo.Lq - 1;
        const bool keys_in_range = c0 + kTile <= geo.kv_len && jfirst >= 0;

        const float sl2 = prm.scale_log2;
        auto stat_index = [&](int i) {
            const int hq = hq0 + i / n_qt;
            const int qr = (qt_lo + i % n_qt) * kTile + ctid;
            return qr < geo.Lq ? ((long long)b * prm.Hq + hq) * geo.Lq + qr : -1ll;
        };
        float lse_next = INFINITY, d_next = 0.f;
        if (n_it > 0) {
            const long long si = stat_index(0);
            if (si >= 0) {
                const float l = prm.LSE[si];
                lse_next = (l == -INFINITY) ? INFINITY : l * kLog2e;
                d_next = prm.Dvec[si];
            }
        }
        const uint64_t sl2x2 = f32x2(sl2, sl2);
        // P^T = 2^(S^T*scale*log2e - LSE_q*log2e) and dS^T = P^T * (dP^T - D_q) for one query tile
        // (query = column); MASKED is a compile-time flag so that full tiles run branch-free code
        auto pt_tile = [&](auto masked_c, const int buf, const int q0) {
            constexpr bool MASKED = decltype(masked_c)::value;
            uint32_t sa_[32], sb_[32], da_[32], db_[32];
            tmem_ld_x32(tSt + lane_off, sa_);
            tmem_ld_x32(tDpt + lane_off, da_);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t(&sv)[32] = (c & 1) ? sb_ : sa_;
                uint32_t(&dv)[32] = (c & 1) ? db_ : da_;
                uint32_t(&sn)[32] = (c & 1) ? sa_ : sb_;
                uint32_t(&dn)[32] = (c & 1) ? da_ : db_;
                tmem_wait_ld_dep(sv);
                tmem_wait_ld_dep(dv);
                if (c < 3) {
                    tmem_ld_x32(tSt + lane_off + (c + 1) * 32, sn);
                    tmem_ld_x32(tDpt + lane_off + (c + 1) * 32, dn);
                }
                uint32_t pk[16], dk[16];
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const float2 l2 = *reinterpret_cast<const float2*>(&s_lse[buf][c * 32 + e]);
                    const float2 dd = *reinterpret_cast<const float2*>(&s_dsum[buf][c * 32 + e]);
                    float t0, t1;
                    f32x2_unpack(fma_f32x2(f32x2_bits(sv[e], sv[e + 1]), sl2x2, f32x2(-l2.x, -l2.y)), t0, t1);
                    float p0 = ex2(t0), p1 = ex2(t1);
                    if (MASKED) {
                        const int q = q0 + c * 32 + e;
                        p0 = (q >= qlo && q <= qhi) ? p0 : 0.f;
                        p1 = (q + 1 >= qlo && q + 1 <= qhi) ? p1 : 0.f;
                    }
                    const uint64_t ds2 = mul_f32x2(f32x2(p0, p1), add_f32x2(f32x2_bits(dv[e], dv[e + 1]), f32x2(-dd.x, -dd.y)));
                    float d0, d1;
                    f32x2_unpack(ds2, d0, d1);
                    pk[e / 2] = pack_bf16(p0, p1);
                    dk[e / 2] = pack_bf16(d0, d1);
                }
                tmem_st_x16(tPt + lane_off + c * 16, pk);
                tmem_st_x16(tDst + lane_off + c * 16, dk);
            }
        };
        bool ok = true;
        for (int i = 0; i < n_it; ++i) {
            const int buf = i & 1;
            s_lse[buf][ctid] = lse_next;
            s_dsum[buf][ctid] = d_next;
            compute_bar_sync();
            lse_next = INFINITY;
            d_next = 0.f;
            if (i + 1 < n_it) {
                const long long si = stat_index(i + 1);
                if (si >= 0) {
                    const float l = prm.LSE[si];
                    lse_next = (l == -INFINITY) ? INFINITY : l * kLog2e;
                    d_next = prm.Dvec[si];
                }
            }
            const int q0 = (qt_lo + i % n_qt) * kTile;
            const bool masked = !(keys_in_range && q0 >= full_qlo && q0 + kTile - 1 <= full_qhi);
            // after a failed wait keep looping (without touching TMEM) so that every compute thread
            // still reaches the named barrier above the same number of times
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull), i & 1, 25));
            if (!ok) continue;
            tc_fence_after();
            if (masked) pt_tile(std::true_type{}, buf, q0);
            else pt_tile(std::false_type{}, buf, q0);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(kBarPFull));
        }
        if (n_it > 0 && ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarDone), 0, 26));
        tc_fence_after();
        const bool row_ok = jl < geo.kv_len;
        __nv_bfloat16* gk = reinterpret_cast<__nv_bfloat16*>(prm.dK) + b * prm.k_stride[0] +
                            (long long)jl * prm.k_stride[1] + slot * prm.k_stride[2];
        __nv_bfloat16* gv = reinterpret_cast<__nv_bfloat16*>(prm.dV) + b * prm.v_stride[0] +
                            (long long)jl * prm.v_stride[1] + slot * prm.v_stride[2];
        if (n_it == 0) {
            if (row_ok)
                for (int e = 0; e < D; e += 8) {
                    *reinterpret_cast<uint4*>(gk + e) = make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(gv + e) = make_uint4(0, 0, 0, 0);
                }
        } else if (ok) {
            const float sc = prm.sm_scale;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t v[32], k[32];
                tmem_ld_x32(tDv + lane_off + c * 32, v);
                tmem_ld_x32(tDk + lane_off + c * 32, k);
                tmem_wait_ld();
                if (row_ok) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
                        o.y = pack_bf16(__uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
                        o.z = pack_bf16(__uint_as_float(v[e + 4]), __uint_as_float(v[e + 5]));
                        o.w = pack_bf16(__uint_as_float(v[e + 6]), __uint_as_float(v[e + 7]));
                        *reinterpret_cast<uint4*>(gv + c * 32 + e) = o;
                        o.x = pack_bf16(__uint_as_float(k[e]) * sc, __uint_as_float(k[e + 1]) * sc);
                        o.y = pack_bf16(__uint_as_float(k[e + 2]) * sc, __uint_as_float(k[e + 3]) * sc);
                        o.z = pack_bf16(__uint_as_float(k[e + 4]) * sc, __uint_as_float(k[e + 5]) * sc);
                        o.w = pack_bf16(__uint_as_float(k[e + 6]) * sc, __uint_as_float(k[e + 7]) * sc);
                        *reinterpret_cast<uint4*>(gk + c * 32 + e) = o;
                    }
                }
            }
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

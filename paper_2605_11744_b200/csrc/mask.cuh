// Segment / tail / past-access mask arithmetic shared by the host-side scheduler and the
// kernels, and the parameter blocks the kernels take.
//
// Global positions: query row r is position p = q_pos0 + r, key row jl is position
// j = kv_pos0 + jl.  With i = p / S and a_i = max(0, i*S - T) (start of the carried tail of
// the previous segment, Section 3.4 "Local Continuity Channel"; C_0 empty, Section 3.1):
//   visible(p, j) <=> lo_vis(p) <= j <= p,  lo_vis(p) = a_i, 0 or i*S by head class   (Appendix C, Eq. "ctx")
//   diff(p, j)    <=> a_i <= j <= p     (reads whose K/V receive gradient; Definition 3.2); i*S <= j <= p
//                     for an own-segment-only head
// For a fixed key j the differentiable queries are also one interval: p in [j, hi_diff(j)),
// hi_diff(j) = end of j's segment, plus the whole next segment when j lies in the last T
// positions of its segment.
#pragma once
#include <cstdint>
#include <cuda.h>

namespace segattn {

constexpr int kTile = 128;     // query rows per tile = key rows per tile
constexpr int kMaxKvHeads = 64;

// Division of a 32-bit unsigned number by a divisor fixed at launch: q = (mulhi(n, m) + n) >> s with
// s = ceil(log2 d), m = floor(2^32 (2^s - d) / d) + 1 (exact for every 32-bit n).  The device's own
// 32-bit division is tens of dependent instructions, and a work item's decode needs several.
struct FastDiv {
    uint32_t d, m, s;
};
inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    if (d == 0) d = 1;  // never used as a divisor then; keeps the fields defined
    uint32_t s = 0;
    while (s < 32 && (1ull << s) < d) ++s;
    f.d = d;
    f.s = s;
    f.m = (uint32_t)((((1ull << s) - d) << 32) / d + 1);
    return f;
}
__host__ __device__ inline uint32_t fdiv(uint32_t n, const FastDiv& f) {
#ifdef __CUDA_ARCH__
    const uint32_t hi = __umulhi(n, f.m);
#else
    const uint32_t hi = (uint32_t)(((unsigned long long)n * f.m) >> 32);
#endif
    return (uint32_t)(((unsigned long long)hi + n) >> f.s);
}

constexpr int kMaxSegs = 256;            // segment starts a call can give (segments of unequal length)
constexpr long long kPosInf = 0x7fffffff;  // "no end": past every supported position

struct MaskGeom {
    FastDiv fS;  // division by S
    int S, T;
    int q_pos0, kv_pos0;
    int Lq, kv_len;
    int detach_before;    // keys before this global position are read forward-only (0: none)
    int flagged_tail_sg;  // flagged heads read the carried tail forward-only too (Appendix C, Eq. "ctx", read literally)
    // Segments of given lengths m_i (Section 3.1) instead of the constant S: n_starts > 0 ascending
    // starts, the first 0, the last segment open-ended.  The carried tail of a segment shorter than T
    // is the whole segment.
    int n_starts;
    int starts[kMaxSegs];
};

// p / S for a non-negative position (positions fit 32 bits: q_pos0 + Lq is limited to 2^30)
__host__ __device__ inline long long seg_of(const MaskGeom& g, long long p) {
    return p <= 0xffffffffLL ? (long long)fdiv((uint32_t)p, g.fS) : p / g.S;
}
// index of the given-length segment that holds position p (n_starts > 0)
__host__ __device__ inline int seg_index(const MaskGeom& g, long long p) {
    int lo = 0, hi = g.n_starts - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (g.starts[mid] <= p) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}
// The given-length forms are kept out of line: they run once per work item, and inlining them into
// the kernels' per-item code costs the constant-length path registers it needs elsewhere.  INL = true
// selects inline copies for code that cannot contain calls (a kernel that re-partitions its register
// file with setmaxnreg).
#if defined(__CUDACC__)
#define SEGATTN_NOINLINE __noinline__
#else
#define SEGATTN_NOINLINE
#endif
__host__ __device__ inline long long seg_start_given_body(const MaskGeom& g, long long p) {
    return (long long)g.starts[seg_index(g, p)];
}
__host__ __device__ inline long long tail_start_given_body(const MaskGeom& g, long long p) {
    const int i = seg_index(g, p);
    const long long prev0 = i > 0 ? g.starts[i - 1] : 0;
    const long long a = (long long)g.starts[i] - g.T;
    return a < prev0 ? prev0 : a;
}
__host__ __device__ SEGATTN_NOINLINE inline long long seg_start_given(const MaskGeom& g, long long p) {
    return seg_start_given_body(g, p);
}
__host__ __device__ SEGATTN_NOINLINE inline long long tail_start_given(const MaskGeom& g, long long p) {
    return tail_start_given_body(g, p);
}
// one past the last reader of key position j (before the detached-prefix rule)
__host__ __device__ SEGATTN_NOINLINE inline long long hi_diff_given(const MaskGeom& g, long long j, bool own_only) {
    const int i = seg_index(g, j);
    const long long e = i + 1 < g.n_starts ? g.starts[i + 1] : kPosInf;
    if (own_only || e == kPosInf || j < e - g.T) return e;
    return i + 2 < g.n_starts ? g.starts[i + 2] : kPosInf;   // a tail position: the next segment reads it too
}
// start of p's segment
template <bool INL = false>
__host__ __device__ inline long long seg_start(const MaskGeom& g, long long p) {
    if (g.n_starts) return INL ? seg_start_given_body(g, p) : seg_start_given(g, p);
    return seg_of(g, p) * (long long)g.S;
}
template <bool INL = false>
__host__ __device__ inline long long tail_start(const MaskGeom& g, long long p) {
    if (g.n_starts) return INL ? tail_start_given_body(g, p) : tail_start_given(g, p);
    long long a = seg_of(g, p) * (long long)g.S - g.T;
    return a < 0 ? 0 : a;
}
// Head classes (Appendix C, Eq. "ctx"): what a KV head's queries read besides their own segment.
constexpr int kHeadLocal = 0;  // the carried tail of the previous segment, differentiably
constexpr int kHeadPast = 1;   // every older position; what lies before the tail start is forward-only
constexpr int kHeadOwn = 2;    // nothing: a long-range head outside the long-range layers
// own segment only on the K/V-gradient side?
__host__ __device__ inline bool diff_own_only(const MaskGeom& g, int cls) {
    return cls == kHeadOwn || (cls == kHeadPast && g.flagged_tail_sg);
}
template <bool INL = false>
__host__ __device__ inline long long lo_visible(const MaskGeom& g, long long p, int cls) {
    if (cls == kHeadPast) return 0;
    return cls == kHeadOwn ? seg_start<INL>(g, p) : tail_start<INL>(g, p);
}
// one past the last query position that differentiably reads key position j of a head of class cls
__host__ __device__ inline long long hi_diff(const MaskGeom& g, long long j, int cls) {
    if (j < g.detach_before) return j;  // no differentiable reader at all
    if (g.n_starts) return hi_diff_given(g, j, diff_own_only(g, cls));
    long long seg_end = (seg_of(g, j) + 1) * (long long)g.S;
    if (diff_own_only(g, cls)) return seg_end;
    return (j >= seg_end - g.T) ? seg_end + g.S : seg_end;
}
// first key position query position p reads differentiably
template <bool INL = false>
__host__ __device__ inline long long lo_diff(const MaskGeom& g, long long p, int cls) {
    const long long lo = diff_own_only(g, cls) ? seg_start<INL>(g, p) : tail_start<INL>(g, p);
    return lo < g.detach_before ? g.detach_before : lo;
}

// Local key-row range [jl_lo, jl_hi] (inclusive) that the query tile starting at row r0 can see;
// empty when jl_hi < jl_lo.
template <bool INL = false>
__host__ __device__ inline void q_tile_kv_range(const MaskGeom& g, int r0, int cls, bool diff_only,
                                                long long* jl_lo, long long* jl_hi) {
    int r_last = r0 + kTile - 1;
    if (r_last > g.Lq - 1) r_last = g.Lq - 1;
    long long p0 = (long long)g.q_pos0 + r0, p1 = (long long)g.q_pos0 + r_last;
    long long lo = diff_only ? lo_diff<INL>(g, p0, cls) : lo_visible<INL>(g, p0, cls);
    long long a = lo - g.kv_pos0, b = p1 - g.kv_pos0;
    if (a < 0) a = 0;
    if (b > g.kv_len - 1) b = g.kv_len - 1;
    *jl_lo = a;
    *jl_hi = b;
}
// Query-row range [r_lo, r_hi] (inclusive) that differentiably reads some key of the key tile
// starting at local row c0; empty when r_hi < r_lo.
__host__ __device__ inline void kv_tile_q_range(const MaskGeom& g, int c0, int cls, long long* r_lo, long long* r_hi) {
    int c_last = c0 + kTile - 1;
    if (c_last > g.kv_len - 1) c_last = g.kv_len - 1;
    long long j0 = (long long)g.kv_pos0 + c0, j1 = (long long)g.kv_pos0 + c_last;
    if (j1 < 0) { *r_lo = 0; *r_hi = -1; return; }
    if (j0 < 0) j0 = 0;
    if (j0 < g.detach_before) j0 = g.detach_before;  // keys before it have no differentiable reader
    if (j0 > j1) { *r_lo = 0; *r_hi = -1; return; }
    long long a = j0 - g.q_pos0;              // first query position is the key itself
    long long b = hi_diff(g, j1, cls) - 1 - g.q_pos0;  // hi_diff is non-decreasing in j
    if (a < 0) a = 0;
    if (b > g.Lq - 1) b = g.Lq - 1;
    *r_lo = a;
    *r_hi = b;
}

// Which KV "slot" (head index inside the K/V tensors handed to the kernel) serves which
// logical KV head, in what launch order, and whether it is flagged.
struct HeadTable {
    uint8_t order[kMaxKvHeads];    // slots sorted heaviest work first: past-access, local, own-segment-only
    uint8_t flag[kMaxKvHeads];     // per slot: head class (kHeadLocal / kHeadPast / kHeadOwn)
    uint8_t logical[kMaxKvHeads];  // per slot: logical KV head (query heads logical*g .. +g-1)
    int n_slots, n_flagged;        // n_flagged: past-access slots (the first n_flagged entries of order)
};

// The work items a persistent CTA takes, in order: the list is sorted heaviest first and dealt to the
// CTAs in rounds, every other round in reverse CTA order, so that no CTA always gets the heaviest item
// of a round.
struct ItemWalk {
    int k, c, G, n;
    __device__ ItemWalk(int cta, int n_ctas, int n_items) : k(0), c(cta), G(n_ctas), n(n_items) {}
    __device__ bool next(int* item) {
        while ((long long)k * G < n) {
            const int i = k * G + ((k & 1) ? G - 1 - c : c);
            ++k;
            if (i < n) {
                *item = i;
                return true;
            }
        }
        return false;
    }
};

struct alignas(64) FwdParams {
    CUtensorMap tq, tk, tv;  // bf16 (d, heads, rows, batch), box (64, 1, 128, 1), 128-byte swizzle
    CUtensorMap to;          // O, for tiled stores
    void* O;
    float* LSE;
    long long o_stride[3];
    MaskGeom geom;
    int B, Hq, g;
    int n_qtiles;
    int n_items;       // work items: B * query heads served * n_qtiles
    FastDiv f_per_f, f_per_u, f_g, f_ncls_f, f_ncls_u;  // divisors of the work-list decode (see fwd_decode)
    float scale_log2;  // sm_scale * log2(e)
    HeadTable heads;
};

struct alignas(64) BwdParams {
    CUtensorMap tq, tk, tv, tdo;  // same form as above
    CUtensorMap tdq, tdk, tdv;    // the gradient tensors, for tiled stores
    const float* LSE;             // [B][Hq][Lq]
    const float* Dvec;            // [B][Hq][Lq]  row dots <dO, O>
    void* dQ;
    void* dK;
    void* dV;
    long long q_stride[3], k_stride[3], v_stride[3];
    MaskGeom geom;
    int B, Hq, Hkv, g;
    int n_qtiles, n_kvtiles;
    int n_items_dq;    // work items of the dQ pass: B * query heads served * n_qtiles
    FastDiv f_per_f, f_per_u, f_g, f_ncls_f, f_ncls_u;  // divisors of the work-list decode (see dq_decode)
    int dkv_tps, dkv_tail_tiles, dkv_n_seg;  // dK/dV grid: key tiles per segment, of which in the tail, segments
    float scale_log2;  // sm_scale * log2(e)
    float sm_scale;
    HeadTable heads;
};

// One work item of the persistent forward and dQ kernels: a 128-row query tile of one (batch, query head).
struct WorkItem {
    int b, hq, slot, qt;
    int cls;  // head class of the item's KV head
};
#if defined(__CUDACC__)
// Decode a position in the work list into a work item, heaviest first: past-access heads (long visible
// ranges) before the others, late query tiles before early ones.  Params is FwdParams or BwdParams.
template <class Params>
__device__ __forceinline__ WorkItem decode_item(const Params& prm, int idx) {
    const HeadTable& ht = prm.heads;
    const int per_f = ht.n_flagged * prm.g * prm.B;
    const int per_u = (ht.n_slots - ht.n_flagged) * prm.g * prm.B;
    const int n_f = per_f * prm.n_qtiles;
    WorkItem it;
    // quotient and remainder through the launch-time reciprocals (the operands are small and non-negative)
    uint32_t q, hb, cls_off, cls_n;
    FastDiv f_cls;
    if (idx < n_f) {
        q = fdiv((uint32_t)idx, prm.f_per_f);
        hb = (uint32_t)idx - q * (uint32_t)per_f;
        cls_off = 0;
        cls_n = (uint32_t)ht.n_flagged;
        f_cls = prm.f_ncls_f;
    } else {
        idx -= n_f;
        q = fdiv((uint32_t)idx, prm.f_per_u);
        hb = (uint32_t)idx - q * (uint32_t)per_u;
        cls_off = (uint32_t)ht.n_flagged;
        cls_n = (uint32_t)(ht.n_slots - ht.n_flagged);
        f_cls = prm.f_ncls_u;
    }
    it.qt = prm.n_qtiles - 1 - (int)q;
    const uint32_t t = fdiv(hb, prm.f_g);
    const uint32_t r = hb - t * (uint32_t)prm.g;
    const uint32_t bb = fdiv(t, f_cls);
    it.slot = ht.order[cls_off + (t - bb * cls_n)];
    it.b = (int)bb;
    it.hq = ht.logical[it.slot] * prm.g + (int)r;
    it.cls = ht.flag[it.slot];
    return it;
}
#endif

}  // namespace segattn

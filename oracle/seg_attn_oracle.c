/*
 * fp64 CPU oracle for segment-level causal attention (forward and its VJP).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA kernels are checked against; nothing on the product path may call it.
 * It shares no code, header, table or helper with the CUDA library.
 *
 * What it computes, in the paper's terms (their T is our L, their M is our T):
 *   - The sequence is cut into non-overlapping segments of constant length S
 *     (Section 3.1 "Setup"; Section 3.5 assumes |x^(i)| = S), or, with seg_starts,
 *     of the lengths m_i the caller gives (Section 3.1 allows them to differ); the
 *     carried tail of a segment shorter than T is the whole segment.
 *   - Each head runs standard scaled dot-product attention
 *     softmax(Q K^T * scale + mask) V over the concatenation [prefix ; segment]
 *     where a segment query sees every prefix position and the within-segment
 *     positions up to and including itself (Appendix C, Eq. "attn").
 *   - The prefix of a local head is the carried KV tail: the last T key/value
 *     vectors of the previous segment, the only differentiable cross-segment
 *     state (Section 3.4 "Local Continuity Channel"; Appendix C, Eq. "ctx").
 *     C_0 is empty, so the first segment is plain causal (Section 3.1).
 *   - A flagged ("past-access") KV head additionally reads older key/values.
 *     Those reads are forward-only: stop-gradient, no gradient path into K/V
 *     (Definition 3.2; Section 3.4 "Long-Range Channel"; Appendix B, Lemma B.1).
 *     Reading taken here: the older past is ALL positions before the tail
 *     start, dense (no top-k retrieval), in union with the tail and the own
 *     segment.  With flagged_tail_is_sg != 0 the flagged head's tail reads are
 *     stop-gradient too (the variant where only local heads carry the state).
 *   - detach_before: in the K-truncated objective the state at the truncation
 *     boundary enters as a constant, sg(C_b) (definition of the K-truncated
 *     consistent objective, Eq. "truncated-base").  A call on a window of
 *     segments passes the global position where its differentiable part starts;
 *     every read of a key before it is stop-gradient: diff additionally
 *     requires j >= detach_before.  0 leaves the mask as stated.
 *   - head_past_mask[c] is a head class: 0 local, 1 flagged as above, 2 a head
 *     whose context is its own segment alone (the long-range head of a layer
 *     outside the long-range layers, Appendix C, Eq. "ctx", third case):
 *     visible = diff = { i*S <= j <= p }.
 *
 * Global positions: query row r sits at p = q_pos0 + r, key row jl at
 * j = kv_pos0 + jl.  With i = p / S and a_i = max(0, i*S - T):
 *     visible(p,j,c) <=> j <= p  and ( j >= a_i  or  flag[c] )
 *     diff(p,j,c)    <=> visible and j >= a_i   (own segment + tail)
 *                        [flagged_tail_is_sg and flag[c]: j >= i*S instead]
 * Forward:  s_j = scale*<q_p,k_j>,  LSE_p = ln sum_j e^{s_j},
 *           P_j = e^{s_j - LSE_p},  O_p = sum_j P_j v_j      over visible j.
 * Backward (softmax VJP, with sg cutting only the K/V side):
 *           D_p = <dO_p,O_p>, dP_j = <dO_p,v_j>, dS_j = P_j (dP_j - D_p),
 *           dQ_p  = scale * sum_{visible j} dS_j k_j,
 *           dK_j += scale * dS_j q_p  and  dV_j += P_j dO_p   only if diff.
 * Query head h uses KV head c = h / (Hq/Hkv); dK/dV sum over the group.
 *
 * Layout: every tensor is contiguous row-major, Q/O/dO/dQ [B][Lq][Hq][d],
 * K/V/dK/dV [B][Lk][Hkv][d], LSE [B][Hq][Lq], all double.
 * Pins: tests/test_oracle_pins.py (library causal attention and autograd,
 * closed forms, finite differences, structural zeros, brute-force counts).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t B, Lq, Lk, Hq, Hkv, d;
    int32_t S, T;
    int32_t q_pos0, kv_pos0;
    int32_t flagged_tail_is_sg;
    int32_t detach_before;   /* keys at global positions below this are read forward-only; 0: none */
    double scale;
    const int32_t *seg_starts; /* NULL: constant length S.  Else n_segs ascending segment starts, the   */
    int32_t n_segs;            /* first 0; segment i = [starts[i], starts[i+1]), the last one open-ended */
} oracle_cfg;

static int cfg_ok(const oracle_cfg *c)
{
    if (c->B < 0 || c->Lq < 0 || c->Lk < 0 || c->Hq <= 0 || c->Hkv <= 0 || c->d <= 0) return 0;
    if (c->Hq % c->Hkv) return 0;
    if (c->seg_starts) {
        if (c->n_segs < 1 || c->seg_starts[0] != 0 || c->T < 0) return 0;
        for (int i = 1; i < c->n_segs; ++i)
            if (c->seg_starts[i] <= c->seg_starts[i - 1]) return 0;
    } else if (c->S <= 0 || c->T < 0 || c->T > c->S) return 0;
    if (c->q_pos0 < 0 || c->detach_before < 0) return 0;
    return 1;
}

/* first visible / first differentiable global key position of query position p */
static void row_bounds(const oracle_cfg *c, int flag, long p, long *lo_vis, long *lo_diff)
{
    long seg0, a;   /* start of p's segment; start of the carried tail of the segment before it */
    if (c->seg_starts) {
        /* segments of lengths m_i (Section 3.1): the tail is the last min(T, m_{i-1}) positions of segment i-1 */
        int i = 0;
        while (i + 1 < c->n_segs && c->seg_starts[i + 1] <= p) ++i;
        seg0 = c->seg_starts[i];
        long prev0 = i > 0 ? c->seg_starts[i - 1] : 0;
        a = seg0 - c->T;
        if (a < prev0) a = prev0;
    } else {
        seg0 = (p / c->S) * (long)c->S;
        a = seg0 - c->T;
    }
    if (a < 0) a = 0;
    if (flag == 2) {             /* own segment only (Appendix C, Eq. "ctx", third case) */
        *lo_vis = *lo_diff = seg0;
    } else {
        *lo_vis = flag ? 0 : a;
        *lo_diff = (flag && c->flagged_tail_is_sg) ? seg0 : a;
    }
    /* the boundary state of a truncated chain is a constant (Eq. "truncated-base"): reads of keys
     * before detach_before carry no gradient into K/V */
    if (*lo_diff < c->detach_before) *lo_diff = c->detach_before;
}

/* One query row: scores, LSE, probabilities P[jl] for jl in [j0,j1) (local key
 * indices), output row.  Returns LSE; p_out must hold Lk doubles. */
static double row_forward(const oracle_cfg *c, const double *q, const double *Kb, const double *Vb,
                          int kvh, long j0, long j1, double *p_out, double *o_out)
{
    const int d = c->d;
    const long kstride = (long)c->Hkv * d;
    double m = -INFINITY;
    for (long jl = j0; jl < j1; ++jl) {
        const double *k = Kb + jl * kstride + (long)kvh * d;
        double s = 0.0;
        for (int e = 0; e < d; ++e) s += q[e] * k[e];
        s *= c->scale;
        p_out[jl] = s;
        if (s > m) m = s;
    }
    double sum = 0.0;
    for (long jl = j0; jl < j1; ++jl) sum += exp(p_out[jl] - m);
    double lse = m + log(sum);
    for (int e = 0; e < d; ++e) o_out[e] = 0.0;
    for (long jl = j0; jl < j1; ++jl) {
        double pj = exp(p_out[jl] - lse);
        p_out[jl] = pj;
        const double *v = Vb + jl * kstride + (long)kvh * d;
        for (int e = 0; e < d; ++e) o_out[e] += pj * v[e];
    }
    return lse;
}

/* local key index range [j0,j1) that global range [lo,p] covers */
static void local_range(const oracle_cfg *c, long lo, long p, long *j0, long *j1)
{
    long a = lo - c->kv_pos0, b = p - c->kv_pos0 + 1;
    if (a < 0) a = 0;
    if (b > c->Lk) b = c->Lk;
    if (b < a) b = a;
    *j0 = a; *j1 = b;
}

int oracle_seg_attn_fwd(const oracle_cfg *c, const double *Q, const double *K, const double *V,
                        const uint8_t *head_past_mask, double *O, double *LSE)
{
    if (!cfg_ok(c)) return 1;
    const int g = c->Hq / c->Hkv, d = c->d;
    const long nrows = (long)c->B * c->Hq * c->Lq;
    int fail = 0;
#pragma omp parallel
    {
        double *pbuf = (double *)malloc(sizeof(double) * (size_t)(c->Lk > 0 ? c->Lk : 1));
        if (!pbuf) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 16)
        for (long idx = 0; idx < nrows; ++idx) {
            if (!pbuf) continue;
            long r = idx % c->Lq;
            int h = (int)((idx / c->Lq) % c->Hq);
            int b = (int)(idx / ((long)c->Lq * c->Hq));
            int kvh = h / g;
            long p = (long)c->q_pos0 + r, lo_vis, lo_diff, j0, j1;
            row_bounds(c, head_past_mask[kvh], p, &lo_vis, &lo_diff);
            local_range(c, lo_vis, p, &j0, &j1);
            const double *q = Q + (((long)b * c->Lq + r) * c->Hq + h) * d;
            double *o = O + (((long)b * c->Lq + r) * c->Hq + h) * d;
            const double *Kb = K + (long)b * c->Lk * c->Hkv * d;
            const double *Vb = V + (long)b * c->Lk * c->Hkv * d;
            double lse;
            if (j1 <= j0) { /* no key present for this row: defined as zeros / -inf */
                for (int e = 0; e < d; ++e) o[e] = 0.0;
                lse = -INFINITY;
            } else {
                lse = row_forward(c, q, Kb, Vb, kvh, j0, j1, pbuf, o);
            }
            LSE[((long)b * c->Hq + h) * c->Lq + r] = lse;
        }
        free(pbuf);
    }
    return fail ? 2 : 0;
}

int oracle_seg_attn_bwd(const oracle_cfg *c, const double *Q, const double *K, const double *V,
                        const double *dO, const uint8_t *head_past_mask,
                        double *dQ, double *dK, double *dV)
{
    if (!cfg_ok(c)) return 1;
    const int g = c->Hq / c->Hkv, d = c->d;
    const long kstride = (long)c->Hkv * d;
    const long nrows = (long)c->B * c->Hq * c->Lq;
    int fail = 0;
    /* per query row: LSE_p and D_p = <dO_p, O_p>, kept for the key-side sums below */
    double *LSE = (double *)malloc(sizeof(double) * (size_t)(nrows > 0 ? nrows : 1));
    double *Dv = (double *)malloc(sizeof(double) * (size_t)(nrows > 0 ? nrows : 1));
    if (!LSE || !Dv) { free(LSE); free(Dv); return 2; }

    /* Query side, one row at a time: dQ_p = scale * sum over visible j of dS_j k_j. */
#pragma omp parallel
    {
        double *pbuf = (double *)malloc(sizeof(double) * (size_t)(c->Lk > 0 ? c->Lk : 1));
        double *orow = (double *)malloc(sizeof(double) * (size_t)d);
        if (!pbuf || !orow) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 16)
        for (long idx = 0; idx < nrows; ++idx) {
            if (!pbuf || !orow) continue;
            long r = idx % c->Lq;
            int h = (int)((idx / c->Lq) % c->Hq);
            int b = (int)(idx / ((long)c->Lq * c->Hq));
            int kvh = h / g;
            long p = (long)c->q_pos0 + r, lo_vis, lo_diff, j0, j1;
            row_bounds(c, head_past_mask[kvh], p, &lo_vis, &lo_diff);
            local_range(c, lo_vis, p, &j0, &j1);
            const double *Kb = K + (long)b * c->Lk * c->Hkv * d;
            const double *Vb = V + (long)b * c->Lk * c->Hkv * d;
            const long qoff = (((long)b * c->Lq + r) * c->Hq + h) * d;
            const double *q = Q + qoff, *go = dO + qoff;
            double *gq = dQ + qoff;
            for (int e = 0; e < d; ++e) gq[e] = 0.0;
            const long sidx = ((long)b * c->Hq + h) * c->Lq + r;
            LSE[sidx] = -INFINITY;
            Dv[sidx] = 0.0;
            if (j1 <= j0) continue;
            LSE[sidx] = row_forward(c, q, Kb, Vb, kvh, j0, j1, pbuf, orow);
            double D = 0.0;
            for (int e = 0; e < d; ++e) D += go[e] * orow[e];
            Dv[sidx] = D;
            for (long jl = j0; jl < j1; ++jl) {
                const double *k = Kb + jl * kstride + (long)kvh * d;
                const double *v = Vb + jl * kstride + (long)kvh * d;
                double dP = 0.0;
                for (int e = 0; e < d; ++e) dP += go[e] * v[e];
                double dS = pbuf[jl] * (dP - D);
                for (int e = 0; e < d; ++e) gq[e] += c->scale * dS * k[e];
            }
        }
        free(pbuf);
        free(orow);
    }

    /* Key side, one key row at a time: sums over the query heads of the group and over the
     * query rows whose read of this key is differentiable (own segment or carried tail);
     * stop-gradient reads contribute nothing. */
    const long nkeys = (long)c->B * c->Lk * c->Hkv;
#pragma omp parallel for schedule(dynamic, 16)
    for (long idx = 0; idx < nkeys; ++idx) {
        int kvh = (int)(idx % c->Hkv);
        long jl = (idx / c->Hkv) % c->Lk;
        int b = (int)(idx / ((long)c->Hkv * c->Lk));
        long j = (long)c->kv_pos0 + jl;
        int flag = head_past_mask[kvh];
        const double *k = K + (((long)b * c->Lk + jl) * c->Hkv + kvh) * d;
        const double *v = V + (((long)b * c->Lk + jl) * c->Hkv + kvh) * d;
        double *gk = dK + (((long)b * c->Lk + jl) * c->Hkv + kvh) * d;
        double *gv = dV + (((long)b * c->Lk + jl) * c->Hkv + kvh) * d;
        for (int e = 0; e < d; ++e) { gk[e] = 0.0; gv[e] = 0.0; }
        if (j < 0) continue;
        for (int h = kvh * g; h < (kvh + 1) * g; ++h) {
            long r_first = j - c->q_pos0;                 /* causal: only rows at or after the key */
            if (r_first < 0) r_first = 0;
            for (long r = r_first; r < c->Lq; ++r) {
                long p = (long)c->q_pos0 + r, lo_vis, lo_diff;
                row_bounds(c, flag, p, &lo_vis, &lo_diff);
                if (j < lo_diff) continue;                /* not visible, or a stop-gradient read */
                const long qoff = (((long)b * c->Lq + r) * c->Hq + h) * d;
                const double *q = Q + qoff, *go = dO + qoff;
                const long sidx = ((long)b * c->Hq + h) * c->Lq + r;
                double s = 0.0, dP = 0.0;
                for (int e = 0; e < d; ++e) { s += q[e] * k[e]; dP += go[e] * v[e]; }
                double P = exp(s * c->scale - LSE[sidx]);
                double dS = P * (dP - Dv[sidx]);
                for (int e = 0; e < d; ++e) {
                    gk[e] += c->scale * dS * q[e];
                    gv[e] += P * go[e];
                }
            }
        }
    }
    free(LSE);
    free(Dv);
    return fail ? 2 : 0;
}

/* Visible / differentiable (query,key) pair counts by direct enumeration of the
 * mask, summed over batch and query heads.  (Cost model of Section 3.5: a local
 * query at in-segment index t of a non-first segment sees t+1+T keys.) */
int oracle_count_pairs(const oracle_cfg *c, const uint8_t *head_past_mask,
                       int64_t *pairs_visible, int64_t *pairs_diff)
{
    if (!cfg_ok(c)) return 1;
    const int g = c->Hq / c->Hkv;
    int64_t nv = 0, nd = 0;
    for (int h = 0; h < c->Hq; ++h) {
        int flag = head_past_mask[h / g];
        for (long r = 0; r < c->Lq; ++r) {
            long p = (long)c->q_pos0 + r, lo_vis, lo_diff, j0, j1;
            row_bounds(c, flag, p, &lo_vis, &lo_diff);
            local_range(c, lo_vis, p, &j0, &j1);
            nv += j1 - j0;
            local_range(c, lo_diff, p, &j0, &j1);
            nd += j1 - j0;
        }
    }
    *pairs_visible = nv * c->B;
    *pairs_diff = nd * c->B;
    return 0;
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

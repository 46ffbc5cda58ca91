// Selection step of the top-k retrieval operator (Appendix D): query summaries, scores against the
// pool, top-k per summary, anchors, window expansion, padding to exactly R positions.  The paper
// states the steps and none of the constants, so every one is a parameter; tie and overflow rules
// are: equal scores go to the lower position, windows are added best anchor first until R positions
// are chosen, and the earliest positions not yet chosen pad a short set.  Floating point decides
// integers here, so the arithmetic is fixed: fp32, products and sums rounded separately, sums taken
// sequentially in index order.  None of this is performance-critical (it runs once per segment and
// reads the pool keys once); the attention over the selected rows is the library's forward.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace segattn {

constexpr int kMaxSummaries = 16;
constexpr int kMaxCandidates = 1024;

struct RetrievalParams {
    const __nv_bfloat16* Q_last;  // [B][Lq_last][Hq][d], contiguous
    const __nv_bfloat16* K_pool;  // strides below (batch, position, head), in elements
    long long pool_stride[3];
    float* summ;      // [B][Hkv][n_sum][d]
    float* scores;    // [B][Hkv][n_sum][P]
    unsigned* mark;   // [B][Hkv][P]: bit m = in summary m's top-k, bit 30 = candidate, bit 31 = selected
    int* picks;       // [B][Hkv][n_sum][top_k]: the top-k picks of each summary, in pick order
    int* idx;         // [B][Hkv][R]
    int B, Hq, Hkv, d, P, Lq_last, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R, n_sum;
};

// step 1: one block per (batch, KV head, summary), one thread per head dimension
__global__ void retrieval_summaries_kernel(const RetrievalParams prm) {
    const int m = blockIdx.x % prm.n_sum;
    const int c = (blockIdx.x / prm.n_sum) % prm.Hkv;
    const int b = blockIdx.x / (prm.n_sum * prm.Hkv);
    const int e = threadIdx.x;
    if (e >= prm.d) return;
    const int g = prm.Hq / prm.Hkv;
    int r0, r1;
    if (m + 1 < prm.n_sum) {  // sliding window m
        r0 = m * prm.stride;
        r1 = r0 + prm.window < prm.Lq_last ? r0 + prm.window : prm.Lq_last;
    } else {                  // the tail average
        r0 = prm.Lq_last - prm.tail > 0 ? prm.Lq_last - prm.tail : 0;
        r1 = prm.Lq_last;
    }
    float acc = 0.f;
    for (int r = 0; r < g; ++r)
        for (int row = r0; row < r1; ++row)
            acc = __fadd_rn(acc, __bfloat162float(prm.Q_last[(((long long)b * prm.Lq_last + row) * prm.Hq + c * g + r) * prm.d + e]));
    prm.summ[(((long long)b * prm.Hkv + c) * prm.n_sum + m) * prm.d + e] = __fdiv_rn(acc, (float)((r1 - r0) * g));
}

// step 2: one thread per pool key; the summaries of the block's (batch, head) sit in shared memory
__global__ void __launch_bounds__(256) retrieval_scores_kernel(const RetrievalParams prm) {
    __shared__ float s_summ[kMaxSummaries * 128];
    const int chunks = (prm.P + 255) / 256;
    const int chunk = blockIdx.x % chunks;
    const int c = (blockIdx.x / chunks) % prm.Hkv;
    const int b = blockIdx.x / (chunks * prm.Hkv);
    const float* summ = prm.summ + ((long long)b * prm.Hkv + c) * prm.n_sum * prm.d;
    for (int i = threadIdx.x; i < prm.n_sum * prm.d; i += 256) s_summ[i] = summ[i];
    __syncthreads();
    const int j = chunk * 256 + threadIdx.x;
    if (j >= prm.P) return;
    const __nv_bfloat16* k = prm.K_pool + b * prm.pool_stride[0] + (long long)j * prm.pool_stride[1] + c * prm.pool_stride[2];
    float acc[kMaxSummaries];
#pragma unroll
    for (int m = 0; m < kMaxSummaries; ++m) acc[m] = 0.f;
    for (int e0 = 0; e0 < prm.d; e0 += 8) {
        const uint4 raw = *reinterpret_cast<const uint4*>(k + e0);
        const __nv_bfloat16* kk = reinterpret_cast<const __nv_bfloat16*>(&raw);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float kv = __bfloat162float(kk[i]);
#pragma unroll
            for (int m = 0; m < kMaxSummaries; ++m)
                if (m < prm.n_sum) acc[m] = __fadd_rn(acc[m], __fmul_rn(s_summ[m * prm.d + e0 + i], kv));
        }
    }
    float* out = prm.scores + ((long long)b * prm.Hkv + c) * prm.n_sum * prm.P;
    for (int m = 0; m < prm.n_sum; ++m) out[(long long)m * prm.P + j] = acc[m];
}

// better of two (score, position) pairs: higher score, then lower position
__device__ __forceinline__ void take_better(float& v, int& j, float v2, int j2) {
    if (v2 > v || (v2 == v && j2 < j)) {
        v = v2;
        j = j2;
    }
}

// step 3: one block per (batch, KV head, summary): top_k block-wide arg-max picks over that summary's
// scores, written in pick order.  Bit m of mark[] is this block's "taken" flag (set atomically: the
// blocks of the other summaries set their own bits in the same words).
__global__ void __launch_bounds__(1024) retrieval_topk_kernel(const RetrievalParams prm) {
    __shared__ float s_v[32];
    __shared__ int s_j[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = blockIdx.x % prm.n_sum;
    const long long bc = blockIdx.x / prm.n_sum;
    const float* sc = prm.scores + (bc * prm.n_sum + m) * prm.P;
    unsigned* mark = prm.mark + bc * prm.P;
    int* picks = prm.picks + (bc * prm.n_sum + m) * prm.top_k;
    for (int t = 0; t < prm.top_k; ++t) {
        float v = -INFINITY;
        int j = 0x7fffffff;
        for (int q = tid; q < prm.P; q += 1024)
            if (!((*reinterpret_cast<volatile unsigned*>(mark + q) >> m) & 1u)) take_better(v, j, sc[q], q);
        for (int o = 16; o > 0; o >>= 1)
            take_better(v, j, __shfl_xor_sync(0xffffffffu, v, o), __shfl_xor_sync(0xffffffffu, j, o));
        if (lane == 0) {
            s_v[warp] = v;
            s_j[warp] = j;
        }
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < 32; ++w) take_better(v, j, s_v[w], s_j[w]);
            picks[t] = j == 0x7fffffff ? -1 : j;
            if (j != 0x7fffffff) atomicOr(mark + j, 1u << m);
        }
        __threadfence_block();
        __syncthreads();
    }
}

// steps 3 (deduplication), 4 and 5: one block per (batch, KV head)
__global__ void __launch_bounds__(256) retrieval_select_kernel(const RetrievalParams prm) {
    __shared__ int s_cand[kMaxCandidates];
    __shared__ float s_cscore[kMaxCandidates];
    __shared__ int s_j[8];
    __shared__ int s_n, s_base;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long bc = blockIdx.x;
    const float* sc = prm.scores + bc * prm.n_sum * prm.P;
    volatile unsigned* mark = prm.mark + bc * prm.P;
    int* idx = prm.idx + bc * prm.R;
    if (tid == 0) {
        // the candidate set, in the order the picks were made (summary by summary)
        const int* picks = prm.picks + bc * prm.n_sum * prm.top_k;
        int n = 0;
        for (int q = 0; q < prm.n_sum * prm.top_k; ++q) {
            const int j = picks[q];
            if (j >= 0 && !(mark[j] & (1u << 30)) && n < kMaxCandidates) {
                mark[j] = mark[j] | (1u << 30);
                s_cand[n++] = j;
            }
        }
        s_n = n;
    }
    __syncthreads();
    // a candidate's score: its best over the summaries
    for (int q = tid; q < s_n; q += 256) {
        float best = -INFINITY;
        for (int m = 0; m < prm.n_sum; ++m) best = fmaxf(best, sc[(long long)m * prm.P + s_cand[q]]);
        s_cscore[q] = best;
    }
    __syncthreads();
    // steps 4 and 5 are a few thousand operations on shared memory: one thread, in the stated order
    if (tid == 0) {
        const int n = s_n;
        int n_sel = 0;
        const int n_anchor = prm.n_anchors < n ? prm.n_anchors : n;
        for (int a = 0; a < n_anchor; ++a) {
            float v = -INFINITY;
            int j = 0x7fffffff, at = -1;
            for (int q = 0; q < n; ++q) {
                if (s_cand[q] < 0) continue;   // already an anchor
                const float v0 = v;
                const int j0 = j;
                take_better(v, j, s_cscore[q], s_cand[q]);
                if (v != v0 || j != j0) at = q;
            }
            if (at < 0) break;
            s_cand[at] = -1;
            for (int p = j - prm.off_lo; p <= j + prm.off_hi; ++p)
                if (p >= 0 && p < prm.P && n_sel < prm.R && !(mark[p] >> 31)) {
                    mark[p] = mark[p] | (1u << 31);
                    ++n_sel;
                }
        }
        for (int p = 0; n_sel < prm.R && p < prm.P; ++p)   // pad with the earliest positions
            if (!(mark[p] >> 31)) {
                mark[p] = mark[p] | (1u << 31);
                ++n_sel;
            }
        s_base = 0;
    }
    __threadfence_block();
    __syncthreads();
    // emit the selected positions in ascending order
    for (int p0 = 0; p0 < prm.P; p0 += 256) {
        const int p = p0 + tid;
        const bool on = p < prm.P && (mark[p] >> 31);
        const unsigned ballot = __ballot_sync(0xffffffffu, on);
        if (lane == 0) s_j[warp] = __popc(ballot);
        __syncthreads();
        int off = s_base;
        for (int w = 0; w < warp; ++w) off += s_j[w];
        if (on) {
            const int at = off + __popc(ballot & ((1u << lane) - 1u));
            if (at < prm.R) idx[at] = p;
        }
        __syncthreads();
        if (tid == 0) {
            int tot = 0;
            for (int w = 0; w < 8; ++w) tot += s_j[w];
            s_base += tot;
        }
        __syncthreads();
    }
}

}  // namespace segattn

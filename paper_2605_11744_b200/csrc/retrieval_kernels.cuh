// Selection step of the top-k retrieval operator (Appendix D): query summaries, scores against the
// pool, top-k per summary, anchors, window expansion, padding to exactly R positions.  The paper
// states the steps and none of the constants, so every one is a parameter; tie and overflow rules
// are: equal scores go to the lower position, windows are added best anchor first until R positions
// are chosen, and the earliest positions not yet chosen pad a short set.  Floating point decides
// integers here, so the arithmetic is fixed: fp32, products and sums rounded separately, sums taken
// sequentially in index order.
//
// The pool keys are read once (that read is the algorithmic traffic, B * Hkv * P * d * 2 bytes); scores are
// never written to memory: a block scores a chunk of 1024 keys in registers and keeps only its own best
// top_k per summary, a second kernel merges the chunks' bests, and the few candidates' scores under the
// other summaries are recomputed where they are needed.  Selected positions live in a bit map.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace segattn {

constexpr int kMaxSummaries = 16;
constexpr int kMaxCandidates = 1024;
constexpr int kRetrKeysPerThread = 4;
constexpr int kRetrChunk = 256 * kRetrKeysPerThread;   // pool keys a block of the scoring kernel takes
constexpr int kRetrSmemWords = 4096;                    // pools up to 128K positions keep their bit map in shared memory

struct RetrievalParams {
    const __nv_bfloat16* Q_last;  // [B][Lq_last][Hq][d], contiguous
    const __nv_bfloat16* K_pool;  // strides below (batch, position, head), in elements
    long long pool_stride[3];
    float* summ;      // [B][Hkv][n_sum][d]
    float* best_v;    // [B][Hkv][n_sum][n_chunks][top_k]: each chunk's best scores per summary, best first
    int* best_j;      //   ... and their positions (-1: the chunk had fewer keys)
    int* picks;       // [B][Hkv][n_sum][top_k]: the top-k picks of each summary, in pick order
    unsigned* bits;   // [B][Hkv][words]: bit p set = position p selected (zeroed before the launch)
    int* idx;         // [B][Hkv][R]
    int B, Hq, Hkv, d, P, Lq_last, window, stride, tail, top_k, n_anchors, off_lo, off_hi, R, n_sum;
    int n_chunks, words;
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
    // the sum runs over (head of the group, row) in that order; loads are issued eight ahead of the ordered adds
    const int n_rows = r1 - r0, n = g * n_rows;
    float acc = 0.f;
    for (int s0 = 0; s0 < n; s0 += 8) {
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int s = s0 + u < n ? s0 + u : n - 1;
            const int r = s / n_rows, row = r0 + s % n_rows;
            v[u] = __bfloat162float(prm.Q_last[(((long long)b * prm.Lq_last + row) * prm.Hq + c * g + r) * prm.d + e]);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (s0 + u < n) acc = __fadd_rn(acc, v[u]);
    }
    prm.summ[(((long long)b * prm.Hkv + c) * prm.n_sum + m) * prm.d + e] = __fdiv_rn(acc, (float)((r1 - r0) * g));
}

// better of two (score, position) pairs: higher score, then lower position
__device__ __forceinline__ void take_better(float& v, int& j, float v2, int j2) {
    if (v2 > v || (v2 == v && j2 < j)) {
        v = v2;
        j = j2;
    }
}
constexpr int kNoPos = 0x7fffffff;

// The best (score, position) pair over a block of 256 threads, returned to every thread.  `buf` alternates
// between calls so that one __syncthreads per call is enough.
__device__ __forceinline__ void block_best(float& v, int& j, float (*s_v)[8], int (*s_j)[8], int buf) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int o = 16; o > 0; o >>= 1)
        take_better(v, j, __shfl_xor_sync(0xffffffffu, v, o), __shfl_xor_sync(0xffffffffu, j, o));
    if (lane == 0) {
        s_v[buf][warp] = v;
        s_j[buf][warp] = j;
    }
    __syncthreads();
    v = s_v[buf][0];
    j = s_j[buf][0];
#pragma unroll
    for (int w = 1; w < 8; ++w) take_better(v, j, s_v[buf][w], s_j[buf][w]);
}

// steps 2 and 3, first half: one block per (batch, KV head, chunk of 1024 pool keys).  A thread scores four
// keys under every summary (the summaries sit in shared memory), then the block picks its top_k per summary
// by top_k rounds of a block-wide arg-max.
template <int NSUM>
__global__ void __launch_bounds__(256) retrieval_score_topk_kernel(const RetrievalParams prm) {
    __shared__ float s_summ[NSUM * 128];
    __shared__ float s_v[2][NSUM][8];
    __shared__ int s_j[2][NSUM][8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk = blockIdx.x % prm.n_chunks;
    const long long bc = blockIdx.x / prm.n_chunks;
    const int c = (int)(bc % prm.Hkv), b = (int)(bc / prm.Hkv);
    const float* summ = prm.summ + bc * prm.n_sum * prm.d;
    for (int i = tid; i < NSUM * prm.d; i += 256) s_summ[i] = i < prm.n_sum * prm.d ? summ[i] : 0.f;
    __syncthreads();
    float acc[kRetrKeysPerThread][NSUM];
    int pos[kRetrKeysPerThread];
    const __nv_bfloat16* kp[kRetrKeysPerThread];
#pragma unroll
    for (int i = 0; i < kRetrKeysPerThread; ++i) {
        pos[i] = chunk * kRetrChunk + i * 256 + tid;
        const int j = pos[i] < prm.P ? pos[i] : prm.P - 1;   // a key past the end is scored but never offered
        kp[i] = prm.K_pool + b * prm.pool_stride[0] + (long long)j * prm.pool_stride[1] + c * prm.pool_stride[2];
#pragma unroll
        for (int m = 0; m < NSUM; ++m) acc[i][m] = 0.f;
    }
    // summaries past n_sum are zero rows: their scores are computed like the others and never read
    uint4 nxt[kRetrKeysPerThread];
#pragma unroll
    for (int i = 0; i < kRetrKeysPerThread; ++i) nxt[i] = *reinterpret_cast<const uint4*>(kp[i]);
    for (int e0 = 0; e0 < prm.d; e0 += 8) {
        uint4 raw[kRetrKeysPerThread];
#pragma unroll
        for (int i = 0; i < kRetrKeysPerThread; ++i) {
            raw[i] = nxt[i];
            if (e0 + 8 < prm.d) nxt[i] = *reinterpret_cast<const uint4*>(kp[i] + e0 + 8);   // in flight during the adds
        }
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            float kv[kRetrKeysPerThread];
#pragma unroll
            for (int i = 0; i < kRetrKeysPerThread; ++i)
                kv[i] = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(&raw[i])[x]);
#pragma unroll
            for (int m = 0; m < NSUM; ++m) {
                const float sv = s_summ[m * prm.d + e0 + x];
#pragma unroll
                for (int i = 0; i < kRetrKeysPerThread; ++i) acc[i][m] = __fadd_rn(acc[i][m], __fmul_rn(sv, kv[i]));
            }
        }
    }
    // top_k rounds; each round picks, for every summary at once, the block's best key not yet taken
    unsigned taken[NSUM];
#pragma unroll
    for (int m = 0; m < NSUM; ++m) {
        taken[m] = 0;
#pragma unroll
        for (int i = 0; i < kRetrKeysPerThread; ++i)
            if (pos[i] >= prm.P) taken[m] |= 1u << i;
    }
    for (int t = 0; t < prm.top_k; ++t) {
        const int buf = t & 1;
        float v[NSUM];
        int j[NSUM];
#pragma unroll
        for (int m = 0; m < NSUM; ++m) {
            v[m] = -INFINITY;
            j[m] = kNoPos;
#pragma unroll
            for (int i = 0; i < kRetrKeysPerThread; ++i)
                if (!((taken[m] >> i) & 1u)) take_better(v[m], j[m], acc[i][m], pos[i]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int m = 0; m < NSUM; ++m)
                take_better(v[m], j[m], __shfl_xor_sync(0xffffffffu, v[m], o), __shfl_xor_sync(0xffffffffu, j[m], o));
        }
        if (lane == 0) {
#pragma unroll
            for (int m = 0; m < NSUM; ++m) {
                s_v[buf][m][warp] = v[m];
                s_j[buf][m][warp] = j[m];
            }
        }
        __syncthreads();
#pragma unroll
        for (int m = 0; m < NSUM; ++m) {
            v[m] = s_v[buf][m][0];
            j[m] = s_j[buf][m][0];
#pragma unroll
            for (int w = 1; w < 8; ++w) take_better(v[m], j[m], s_v[buf][m][w], s_j[buf][m][w]);
#pragma unroll
            for (int i = 0; i < kRetrKeysPerThread; ++i)
                if (pos[i] == j[m]) taken[m] |= 1u << i;
        }
        if (tid < prm.n_sum) {
            // thread m writes summary m's pick of this round
            float vm = v[0];
            int jm = j[0];
#pragma unroll
            for (int m = 1; m < NSUM; ++m)
                if (tid == m) {
                    vm = v[m];
                    jm = j[m];
                }
            const long long at = ((bc * prm.n_sum + tid) * prm.n_chunks + chunk) * prm.top_k + t;
            prm.best_v[at] = vm;
            prm.best_j[at] = jm == kNoPos ? -1 : jm;
        }
    }
}

// step 3, second half: one block per (batch, KV head, summary) merges the chunks' bests into the summary's
// top_k picks, best first.
__global__ void __launch_bounds__(256) retrieval_merge_kernel(const RetrievalParams prm) {
    __shared__ float s_v[2][8];
    __shared__ int s_j[2][8];
    constexpr int kHeld = 16;           // entries a thread keeps in registers (covers pools of 256K positions at top_k = 16)
    const int tid = threadIdx.x;
    const long long bcm = blockIdx.x;   // (batch, head, summary)
    const int n = prm.n_chunks * prm.top_k;
    const float* in_v = prm.best_v + bcm * n;
    const int* in_j = prm.best_j + bcm * n;
    int* picks = prm.picks + bcm * prm.top_k;
    float hv[kHeld];
    int hj[kHeld];
#pragma unroll
    for (int u = 0; u < kHeld; ++u) {
        const int q = tid + u * 256;
        hj[u] = q < n ? in_j[q] : -1;
        hv[u] = q < n ? in_v[q] : -INFINITY;
    }
    int last = kNoPos;   // the position picked in the previous round
    float last_v = INFINITY;
    for (int t = 0; t < prm.top_k; ++t) {
        // the best entry that comes after the previous pick in the order (score descending, position ascending):
        // entries are distinct positions, so "after" is a strict comparison and nothing has to be marked
        float v = -INFINITY;
        int j = kNoPos;
        auto offer = [&](float vq, int jq) {
            if (jq < 0) return;
            const bool after = t == 0 || vq < last_v || (vq == last_v && jq > last);
            if (after) take_better(v, j, vq, jq);
        };
#pragma unroll
        for (int u = 0; u < kHeld; ++u) offer(hv[u], hj[u]);
        for (int q = tid + kHeld * 256; q < n; q += 256) offer(in_v[q], in_j[q]);   // what the registers do not hold
        block_best(v, j, s_v, s_j, t & 1);
        if (tid == 0) picks[t] = j == kNoPos ? -1 : j;
        if (j == kNoPos) {   // fewer than top_k keys in the pool: the rest stays empty
            for (int u = t + 1 + tid; u < prm.top_k; u += 256) picks[u] = -1;
            break;
        }
        last = j;
        last_v = v;
    }
}

// inclusive prefix sum of one int per thread over a block of 256 threads; *total gets the block's sum
__device__ __forceinline__ int block_scan_incl(int x, int* s_w, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    __syncthreads();   // s_w may still be read from a previous call
    if (lane == 31) s_w[warp] = x;
    __syncthreads();
    int off = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        if (w < warp) off += s_w[w];
        tot += s_w[w];
    }
    *total = tot;
    return x + off;
}

// steps 3 (deduplication), 4 and 5: one block per (batch, KV head)
__global__ void __launch_bounds__(256) retrieval_select_kernel(const RetrievalParams prm) {
    extern __shared__ float s_summ[];               // [n_sum][d]
    __shared__ int s_cand[kMaxCandidates];
    __shared__ float s_cscore[kMaxCandidates];
    __shared__ float s_v[2][8];
    __shared__ int s_j[2][8];
    __shared__ int s_w[8];
    __shared__ unsigned s_bits[kRetrSmemWords];   // the bit map of selected positions, when the pool is small enough
    const int tid = threadIdx.x;
    const long long bc = blockIdx.x;
    const int c = (int)(bc % prm.Hkv), b = (int)(bc / prm.Hkv);
    const float* summ = prm.summ + bc * prm.n_sum * prm.d;
    for (int i = tid; i < prm.n_sum * prm.d; i += 256) s_summ[i] = summ[i];
    // larger pools use the (zeroed) bit map in the workspace; both are only ever touched by this block
    unsigned* bits = prm.words <= kRetrSmemWords ? s_bits : prm.bits + bc * prm.words;
    if (prm.words <= kRetrSmemWords)
        for (int i = tid; i < prm.words; i += 256) s_bits[i] = 0u;
    // the candidate set, in the order the picks were made (summary by summary): a pick is dropped when the same
    // position was picked earlier
    const int* picks = prm.picks + bc * prm.n_sum * prm.top_k;
    const int n_picks = prm.n_sum * prm.top_k;    // <= kMaxCandidates
    int n_cand = 0;
    for (int q0 = 0; q0 < n_picks; q0 += 256) {
        const int q = q0 + tid;
        int j = q < n_picks ? picks[q] : -1;
        if (j >= 0)
            for (int u = 0; u < q; ++u)
                if (picks[u] == j) {
                    j = -1;
                    break;
                }
        int tot;
        const int at = block_scan_incl(j >= 0 ? 1 : 0, s_w, &tot);
        if (j >= 0) s_cand[n_cand + at - 1] = j;
        n_cand += tot;
    }
    __syncthreads();
    // a candidate's score: its best over the summaries (recomputed: scores are not kept in memory)
    for (int q = tid; q < n_cand; q += 256) {
        const __nv_bfloat16* k = prm.K_pool + b * prm.pool_stride[0] + (long long)s_cand[q] * prm.pool_stride[1] +
                                 c * prm.pool_stride[2];
        uint4 row[16];   // the key row, read once (d <= 128)
#pragma unroll
        for (int u = 0; u < 16; ++u)
            if (u * 8 < prm.d) row[u] = *reinterpret_cast<const uint4*>(k + u * 8);
        float best = -INFINITY;
        for (int m = 0; m < prm.n_sum; ++m) {
            const float* sm = s_summ + m * prm.d;
            float acc = 0.f;
#pragma unroll
            for (int u = 0; u < 16; ++u)
                if (u * 8 < prm.d) {
                    const __nv_bfloat16* kk = reinterpret_cast<const __nv_bfloat16*>(&row[u]);
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc = __fadd_rn(acc, __fmul_rn(sm[u * 8 + i], __bfloat162float(kk[i])));
                }
            best = fmaxf(best, acc);
        }
        s_cscore[q] = best;
    }
    __syncthreads();
    // steps 4 and 5: anchors best first; each adds the positions of its window that are in range and not yet
    // selected, in ascending order, while fewer than R are selected
    const int n_anchor = prm.n_anchors < n_cand ? prm.n_anchors : n_cand;
    const int W = prm.off_lo + prm.off_hi + 1;
    int n_sel = 0;
    for (int a = 0; a < n_anchor && n_sel < prm.R; ++a) {
        float v = -INFINITY;
        int j = kNoPos;
        for (int q = tid; q < n_cand; q += 256)
            if (s_cand[q] >= 0) take_better(v, j, s_cscore[q], s_cand[q]);
        block_best(v, j, s_v, s_j, a & 1);
        for (int q = tid; q < n_cand; q += 256)
            if (s_cand[q] == j) s_cand[q] = -1;   // used as an anchor
        for (int w0 = 0; w0 < W && n_sel < prm.R; w0 += 256) {
            const int p = j - prm.off_lo + w0 + tid;
            const bool fresh = w0 + tid < W && p >= 0 && p < prm.P &&
                               !((*reinterpret_cast<volatile unsigned*>(bits + (p >> 5)) >> (p & 31)) & 1u);
            int tot;
            const int rank = block_scan_incl(fresh ? 1 : 0, s_w, &tot);   // 1-based among the fresh ones
            if (fresh && n_sel + rank <= prm.R) atomicOr(bits + (p >> 5), 1u << (p & 31));
            n_sel += tot < prm.R - n_sel ? tot : prm.R - n_sel;
            __threadfence_block();
            __syncthreads();
        }
    }
    // pad with the earliest positions not yet selected
    for (int w0 = 0; w0 < prm.words && n_sel < prm.R; w0 += 256) {
        const int w = w0 + tid;
        unsigned word = 0xffffffffu, valid = 0;
        if (w < prm.words) {
            word = *reinterpret_cast<volatile unsigned*>(bits + w);
            const int left = prm.P - w * 32;
            valid = left >= 32 ? 0xffffffffu : (1u << left) - 1u;
        }
        const unsigned zeros = ~word & valid;
        int tot;
        const int incl = block_scan_incl(__popc(zeros), s_w, &tot);
        const int before = incl - __popc(zeros), need = prm.R - n_sel;
        if (zeros && before < need) {
            unsigned add = zeros;
            if (before + __popc(zeros) > need) {   // only the lowest (need - before) unselected positions of this word
                add = 0;
                unsigned z = zeros;
                for (int k = 0; k < need - before; ++k) {
                    add |= z & (0u - z);
                    z &= z - 1;
                }
            }
            bits[w] = word | add;
        }
        n_sel += tot < need ? tot : need;
        __syncthreads();
    }
    __threadfence_block();
    __syncthreads();
    // emit the selected positions in ascending order
    int* idx = prm.idx + bc * prm.R;
    int base = 0;
    for (int w0 = 0; w0 < prm.words; w0 += 256) {
        const int w = w0 + tid;
        unsigned word = w < prm.words ? *reinterpret_cast<volatile unsigned*>(bits + w) : 0u;
        int tot;
        int at = base + block_scan_incl(__popc(word), s_w, &tot) - __popc(word);
        while (word) {
            const int bit = __ffs(word) - 1;
            if (at < prm.R) idx[at] = w * 32 + bit;
            ++at;
            word &= word - 1;
        }
        base += tot;
    }
}

}  // namespace segattn

// Data movement of the streamed prefill (the segment recurrence of Definition 3.1): append one
// segment's K/V to the retained state, and carry the last T positions over as the next tail
// (Section 3.4: past-only pool for flagged heads, carried KV tail for the others).
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace segattn {

struct PrefillCopyParams {
    const uint4* Kseg;  // [B][S][Hkv][d] (strides in 16-byte units below)
    const uint4* Vseg;
    uint4* Kpool;       // [B][n_flag][Lmax][d]
    uint4* Vpool;
    uint4* Kwin;        // [B][n_unflag][T+S][d]: rows [0,T) previous tail, rows [T,T+S) current segment
    uint4* Vwin;
    long long seg_stride[3];  // (batch, position, head) of Kseg/Vseg, in uint4 units
    int B, S, T, Hkv, Lmax, n_flag, n_unflag;
    int rows;           // rows of the incoming segment (S, or fewer for a shorter segment)
    int d16;            // d * 2 / 16: uint4 per head row
    int pos0;           // first global position of this segment
    uint8_t slot_of_head[64];  // KV head -> slot inside its class (pool slot or window slot)
    uint8_t flag_of_head[64];
};

// one thread per 16 bytes of the incoming segment (K and V both)
__global__ void __launch_bounds__(256) prefill_append_kernel(const PrefillCopyParams prm) {
    const long long n = (long long)prm.B * prm.rows * prm.Hkv * prm.d16;
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= n) return;
    const int e = (int)(idx % prm.d16);
    const int h = (int)((idx / prm.d16) % prm.Hkv);
    const int r = (int)((idx / ((long long)prm.d16 * prm.Hkv)) % prm.rows);
    const int b = (int)(idx / ((long long)prm.d16 * prm.Hkv * prm.rows));
    const long long src = b * prm.seg_stride[0] + (long long)r * prm.seg_stride[1] + h * prm.seg_stride[2] + e;
    const uint4 k = prm.Kseg[src], v = prm.Vseg[src];
    const int slot = prm.slot_of_head[h];
    if (prm.flag_of_head[h]) {
        const long long dst = (((long long)b * prm.n_flag + slot) * prm.Lmax + prm.pos0 + r) * prm.d16 + e;
        prm.Kpool[dst] = k;
        prm.Vpool[dst] = v;
    } else {
        const long long dst = (((long long)b * prm.n_unflag + slot) * (prm.T + prm.S) + prm.T + r) * prm.d16 + e;
        prm.Kwin[dst] = k;
        prm.Vwin[dst] = v;
    }
}

// The carried tail: window rows [src_row, src_row + n_rows) (the last positions of the segment just processed)
// -> rows [dst_row, dst_row + n_rows), which end at row T where the next segment begins.  The two ranges never
// overlap (the source starts at row T or later).  `pitch` = T + S rows per (batch, head) unit.
__global__ void __launch_bounds__(256) prefill_roll_tail_kernel(uint4* Kwin, uint4* Vwin, int n_units, int pitch,
                                                                int src_row, int dst_row, int n_rows, int d16) {
    const long long per = (long long)n_rows * d16;
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= per * n_units) return;
    const long long u = idx / per, off = idx % per;
    const long long base = u * (long long)pitch * d16;
    Kwin[base + (long long)dst_row * d16 + off] = Kwin[base + (long long)src_row * d16 + off];
    Vwin[base + (long long)dst_row * d16 + off] = Vwin[base + (long long)src_row * d16 + off];
}

// Gradients of the streamed backward, from the two per-class scratch tensors ([B][n][T+S][d], slot order)
// to the caller's [B][T+S][Hkv][d]: one thread per 16 bytes (dK and dV both).
__global__ void __launch_bounds__(256) prefill_scatter_grads_kernel(const PrefillCopyParams prm, const uint4* gKf,
                                                                    const uint4* gVf, const uint4* gKu, const uint4* gVu,
                                                                    uint4* dK, uint4* dV) {
    const int rows = prm.T + prm.S;
    const long long n = (long long)prm.B * rows * prm.Hkv * prm.d16;
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= n) return;
    const int e = (int)(idx % prm.d16);
    const int h = (int)((idx / prm.d16) % prm.Hkv);
    const int r = (int)((idx / ((long long)prm.d16 * prm.Hkv)) % rows);
    const int b = (int)(idx / ((long long)prm.d16 * prm.Hkv * rows));
    const int slot = prm.slot_of_head[h];
    if (prm.flag_of_head[h]) {
        const long long src = (((long long)b * prm.n_flag + slot) * rows + r) * prm.d16 + e;
        dK[idx] = gKf[src];
        dV[idx] = gVf[src];
    } else {
        const long long src = (((long long)b * prm.n_unflag + slot) * rows + r) * prm.d16 + e;
        dK[idx] = gKu[src];
        dV[idx] = gVu[src];
    }
}

// Context of a head that reads a retrieved prefix (Appendix C, Eq. "ctx", first case): rows [0, R) of
// the output are the pool rows the index list names, rows [R, R + Lseg) the current segment's.  One
// thread per 16 bytes of output (K and V both).  An index outside [0, pool_len) gives a zero row and
// sets the status word (code 1, invalid input) instead of reading out of bounds.
struct GatherParams {
    const uint4* Kpool;  // strides below, in uint4 units, for (batch, position, head)
    const uint4* Vpool;
    const uint4* Kseg;
    const uint4* Vseg;
    const int32_t* idx;  // [B][Hkv][R]
    uint4* Kctx;         // [B][R + Lseg][Hkv][d], contiguous
    uint4* Vctx;
    long long pool_stride[3], seg_stride[3];
    int B, Hkv, R, Lseg, pool_len;
    int d16;             // d * 2 / 16
};
__global__ void __launch_bounds__(256) gather_context_kernel(const GatherParams prm, int* status) {
    const int rows = prm.R + prm.Lseg;
    const long long n = (long long)prm.B * rows * prm.Hkv * prm.d16;
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    const int e = (int)(i % prm.d16);
    const int h = (int)((i / prm.d16) % prm.Hkv);
    const int r = (int)((i / ((long long)prm.d16 * prm.Hkv)) % rows);
    const int b = (int)(i / ((long long)prm.d16 * prm.Hkv * rows));
    uint4 k = make_uint4(0, 0, 0, 0), v = k;
    if (r < prm.R) {
        const int j = prm.idx[((long long)b * prm.Hkv + h) * prm.R + r];
        if (j >= 0 && j < prm.pool_len) {
            const long long src = b * prm.pool_stride[0] + (long long)j * prm.pool_stride[1] + h * prm.pool_stride[2] + e;
            k = prm.Kpool[src];
            v = prm.Vpool[src];
        } else if (e == 0) {
            atomicCAS(status, 0, (1 << 8) | 1);
        }
    } else {
        const long long src = b * prm.seg_stride[0] + (long long)(r - prm.R) * prm.seg_stride[1] + h * prm.seg_stride[2] + e;
        k = prm.Kseg[src];
        v = prm.Vseg[src];
    }
    prm.Kctx[i] = k;
    prm.Vctx[i] = v;
}

}  // namespace segattn

// Rotary position embedding with re-indexed positions (Section 3.4 "RoPE Re-indexing for Prefix
// Concatenation", Appendix E): a prefix of P rows put in front of a segment is rotated with positions
// 0..P-1, the segment's queries and keys with P..P+m-1, values stay as they are.  The rotation acts on
// the pairs (x[i], x[i + d/2]) with angle pos * base^(-2i/d).  All three kernels are plain streams over
// HBM: 16-byte loads and stores, the cos/sin table (a few MB at most, shared by every head and batch
// element) served by L2.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace segattn {

// table[pos][i] = (cos, sin)(pos * base^(-2i/d)), i < d/2, in double precision rounded once to fp32
__global__ void __launch_bounds__(256) rope_table_kernel(float2* table, int n_pos, int half_d, double base) {
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= (long long)n_pos * half_d) return;
    const int f = (int)(i % half_d);
    const int pos = (int)(i / half_d);
    const double inv_freq = pow(base, -(double)f / (double)half_d);   // base^(-2f/d)
    double s, c;
    sincos((double)pos * inv_freq, &s, &c);
    table[i] = make_float2((float)c, (float)s);
}

// Rotates the eight pairs (lo[k], hi[k]) by the table entries cs[k]; sign = -1 rotates back.
__device__ __forceinline__ void rope_rotate8(uint4& lo, uint4& hi, const float2* __restrict__ cs, float sign) {
    const float4* t4 = reinterpret_cast<const float4*>(cs);
    __nv_bfloat162* l2 = reinterpret_cast<__nv_bfloat162*>(&lo);
    __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&hi);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float4 t = t4[k];                      // (cos, sin) of elements 2k and 2k+1
        const float2 a = __bfloat1622float2(l2[k]), b = __bfloat1622float2(h2[k]);
        const float s0 = sign * t.y, s1 = sign * t.w;
        const float y0 = fmaf(a.x, t.x, -b.x * s0), z0 = fmaf(a.x, s0, b.x * t.x);
        const float y1 = fmaf(a.y, t.z, -b.y * s1), z1 = fmaf(a.y, s1, b.y * t.z);
        l2[k] = __floats2bfloat162_rn(y0, y1);
        h2[k] = __floats2bfloat162_rn(z0, z1);
    }
}

// Y[b][r][h][:] = Rot(+-(pos0 + r)) X[b][r][h][:].  One thread per 16 bytes of the lower half of a head row
// and the 16 bytes it pairs with in the upper half.  Strides in elements for (batch, row, head).
struct RopeApplyParams {
    const __nv_bfloat16* X;
    __nv_bfloat16* Y;
    const float2* table;  // [n_pos][d/2]
    long long x_stride[3], y_stride[3];
    int B, L, H, d, pos0;
    float sign;
};
__global__ void __launch_bounds__(256) rope_apply_kernel(const RopeApplyParams prm) {
    const int per_row = prm.d / 16;   // threads per head row
    const long long n = (long long)prm.B * prm.L * prm.H * per_row;
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    const int e = (int)(i % per_row) * 8;
    const int h = (int)((i / per_row) % prm.H);
    const int r = (int)((i / ((long long)per_row * prm.H)) % prm.L);
    const int b = (int)(i / ((long long)per_row * prm.H * prm.L));
    const __nv_bfloat16* x = prm.X + b * prm.x_stride[0] + (long long)r * prm.x_stride[1] + h * prm.x_stride[2];
    __nv_bfloat16* y = prm.Y + b * prm.y_stride[0] + (long long)r * prm.y_stride[1] + h * prm.y_stride[2];
    uint4 lo = *reinterpret_cast<const uint4*>(x + e), hi = *reinterpret_cast<const uint4*>(x + prm.d / 2 + e);
    rope_rotate8(lo, hi, prm.table + (long long)(prm.pos0 + r) * (prm.d / 2) + e, prm.sign);
    *reinterpret_cast<uint4*>(y + e) = lo;
    *reinterpret_cast<uint4*>(y + prm.d / 2 + e) = hi;
}

// [K_ret ; K_i] with re-indexed rotations and [V_ret ; V_i] unrotated, from an index list: row r < R of the
// output is pool row idx[b][h][r] rotated by position r, row R + t is segment row t rotated by R + t.  An
// index outside [0, pool_len) gives a zero row and sets the status word, as in the plain gather.
struct GatherRopeParams {
    const __nv_bfloat16* Kpool;  // element strides below for (batch, position, head)
    const __nv_bfloat16* Vpool;
    const __nv_bfloat16* Kseg;
    const __nv_bfloat16* Vseg;
    const int32_t* idx;          // [B][Hkv][R]
    __nv_bfloat16* Kctx;         // [B][R + Lseg][Hkv][d], contiguous
    __nv_bfloat16* Vctx;
    const float2* table;         // [n_pos >= R + Lseg][d/2]
    long long pool_stride[3], seg_stride[3];
    int B, Hkv, R, Lseg, pool_len, d;
};
__global__ void __launch_bounds__(256) gather_context_rope_kernel(const GatherRopeParams prm, int* status) {
    const int rows = prm.R + prm.Lseg;
    const int per_row = prm.d / 16;
    const long long n = (long long)prm.B * rows * prm.Hkv * per_row;
    const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    const int e = (int)(i % per_row) * 8;
    const int h = (int)((i / per_row) % prm.Hkv);
    const int r = (int)((i / ((long long)per_row * prm.Hkv)) % rows);
    const int b = (int)(i / ((long long)per_row * prm.Hkv * rows));
    const __nv_bfloat16 *k = nullptr, *v = nullptr;
    if (r < prm.R) {
        const int j = prm.idx[((long long)b * prm.Hkv + h) * prm.R + r];
        if (j >= 0 && j < prm.pool_len) {
            const long long src = b * prm.pool_stride[0] + (long long)j * prm.pool_stride[1] + h * prm.pool_stride[2];
            k = prm.Kpool + src;
            v = prm.Vpool + src;
        } else if (e == 0) {
            atomicCAS(status, 0, (1 << 8) | 1);
        }
    } else {
        const long long src = b * prm.seg_stride[0] + (long long)(r - prm.R) * prm.seg_stride[1] + h * prm.seg_stride[2];
        k = prm.Kseg + src;
        v = prm.Vseg + src;
    }
    const int half = prm.d / 2;
    uint4 klo = make_uint4(0, 0, 0, 0), khi = klo, vlo = klo, vhi = klo;
    if (k) {
        klo = *reinterpret_cast<const uint4*>(k + e);
        khi = *reinterpret_cast<const uint4*>(k + half + e);
        vlo = *reinterpret_cast<const uint4*>(v + e);
        vhi = *reinterpret_cast<const uint4*>(v + half + e);
        rope_rotate8(klo, khi, prm.table + (long long)r * half + e, 1.f);
    }
    const long long dst = (((long long)b * rows + r) * prm.Hkv + h) * prm.d;
    *reinterpret_cast<uint4*>(prm.Kctx + dst + e) = klo;
    *reinterpret_cast<uint4*>(prm.Kctx + dst + half + e) = khi;
    *reinterpret_cast<uint4*>(prm.Vctx + dst + e) = vlo;
    *reinterpret_cast<uint4*>(prm.Vctx + dst + half + e) = vhi;
}

}  // namespace segattn

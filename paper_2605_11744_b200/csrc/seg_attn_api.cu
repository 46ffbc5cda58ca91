// C ABI of the library (see include/seg_attn.h): argument validation, tensor-map construction,
// the host side of the mask scheduler, and kernel launches.  Built as one translation unit.
#include "seg_attn.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include <cuda.h>
#include <cuda_runtime.h>

#include "bwd_kernels.cuh"
#include "fwd_kernel.cuh"
#include "mask.cuh"
#include "prefill_kernels.cuh"
#include "retrieval_kernels.cuh"
#include "rope_kernels.cuh"

using namespace segattn;

namespace {

thread_local int t_last_cuda_error = 0;
std::atomic<long long> g_launches{0};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime so that the library does not
// link against libcuda (it must load on machines without a driver).
EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// SEGATTN_LOG=1 in the environment: one line per launch on stderr with the shapes and the schedule's size.
bool log_on() {
    static const bool on = [] {
        const char* v = getenv("SEGATTN_LOG");
        return v && *v && *v != '0';
    }();
    return on;
}

segattn_status cuda_fail(cudaError_t e) {
    t_last_cuda_error = (int)e;
    return SEGATTN_ERR_CUDA;
}

segattn_status check_arch() {
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    return major == 10 ? SEGATTN_OK : SEGATTN_ERR_UNSUPPORTED_ARCH;
}

// number of SMs of the current device
segattn_status sm_count(int* n) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaDeviceGetAttribute(n, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    return *n > 0 ? SEGATTN_OK : SEGATTN_ERR_CUDA;
}

bool strides_ok(const int64_t s[3], int d) {
    (void)d;
    for (int i = 0; i < 3; ++i)
        if (s[i] < 0 || (s[i] % 8) != 0) return false;
    return true;
}

bool params_ok(const seg_attn_params* p) {
    if (!p) return false;
    if (p->B < 0 || p->Lq < 0 || p->kv_len < 0) return false;
    if (p->Hq <= 0 || p->Hkv <= 0 || p->Hkv > kMaxKvHeads || p->Hq % p->Hkv) return false;
    if (p->d != 64 && p->d != 128) return false;
    if (p->S < 1 || p->T < 0) return false;
    if (p->seg_starts) {
        if (p->n_segs < 1 || p->n_segs > kMaxSegs || p->seg_starts[0] != 0) return false;
        for (int i = 1; i < p->n_segs; ++i)
            if (p->seg_starts[i] <= p->seg_starts[i - 1]) return false;
    } else if (p->T > p->S) {
        return false;
    }
    if (p->q_pos0 < 0 || p->detach_before < 0) return false;
    if (p->flags & ~SEGATTN_FLAG_FLAGGED_TAIL_SG) return false;
    if (!(p->sm_scale > 0.f) || !std::isfinite(p->sm_scale)) return false;
    if ((long long)p->q_pos0 + p->Lq > 0x7fffffffLL / 2) return false;
    return true;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// bf16 tensor viewed as (d, heads, rows, batch); box = 64 columns x 128 rows, 128-byte swizzle.
segattn_status make_map(CUtensorMap* m, const void* base, int d, int heads, long long rows, int batch,
                        const int64_t stride[3]) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) {
        t_last_cuda_error = (int)cudaErrorSymbolNotFound;
        return SEGATTN_ERR_CUDA;
    }
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)heads, (cuuint64_t)(rows > 0 ? rows : 1),
                          (cuuint64_t)(batch > 0 ? batch : 1)};
    // a stride of a size-1 dimension is never used for addressing but must still be valid
    auto bytes = [&](int64_t s) { return (cuuint64_t)((s > 0 ? s : d) * 2); };
    cuuint64_t strides[3] = {bytes(stride[2]), bytes(stride[1]), bytes(stride[0])};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)kTile, 1};
    cuuint32_t elem[4] = {1, 1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, elem,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        t_last_cuda_error = (int)r;
        return SEGATTN_ERR_CUDA;
    }
    return SEGATTN_OK;
}

// every entry of the per-KV-head class array is one of SEGATTN_HEAD_LOCAL / _PAST / _OWN
bool mask_ok(const uint8_t* mask, int Hkv) {
    if (!mask) return false;
    for (int c = 0; c < Hkv; ++c)
        if (mask[c] > SEGATTN_HEAD_OWN) return false;
    return true;
}

void identity_heads(HeadTable* ht, int Hkv, const uint8_t* mask) {
    ht->n_slots = Hkv;
    int k = 0;
    // launch order: heaviest class first (past-access, then local, then own-segment-only)
    const int by_weight[3] = {kHeadPast, kHeadLocal, kHeadOwn};
    for (int w = 0; w < 3; ++w) {
        for (int c = 0; c < Hkv; ++c)
            if (mask[c] == by_weight[w]) ht->order[k++] = (uint8_t)c;
        if (w == 0) ht->n_flagged = k;
    }
    for (int c = 0; c < Hkv; ++c) {
        ht->flag[c] = mask[c];
        ht->logical[c] = (uint8_t)c;
    }
}

// launch-time reciprocals of the work-list decode (fwd_decode / dq_decode)
template <class Params>
void set_decode_divisors(Params& prm, const HeadTable& ht, int g, int B) {
    prm.f_per_f = make_fastdiv((uint32_t)(ht.n_flagged * g * B));
    prm.f_per_u = make_fastdiv((uint32_t)((ht.n_slots - ht.n_flagged) * g * B));
    prm.f_g = make_fastdiv((uint32_t)g);
    prm.f_ncls_f = make_fastdiv((uint32_t)ht.n_flagged);
    prm.f_ncls_u = make_fastdiv((uint32_t)(ht.n_slots - ht.n_flagged));
}

MaskGeom geom_of(const seg_attn_params* p) {
    MaskGeom g;
    g.fS = make_fastdiv((uint32_t)p->S);
    g.S = p->S;
    g.T = p->T;
    g.q_pos0 = p->q_pos0;
    g.kv_pos0 = p->kv_pos0;
    g.Lq = p->Lq;
    g.kv_len = p->kv_len;
    g.flagged_tail_sg = (p->flags & SEGATTN_FLAG_FLAGGED_TAIL_SG) ? 1 : 0;
    g.detach_before = p->detach_before;
    g.n_starts = p->seg_starts ? p->n_segs : 0;
    for (int i = 0; i < kMaxSegs; ++i) g.starts[i] = i < g.n_starts ? p->seg_starts[i] : 0;
    return g;
}

template <typename K>
segattn_status set_smem(K kernel, int bytes) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e == cudaSuccess ? SEGATTN_OK : cuda_fail(e);
}

segattn_status launch_check() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
    g_launches.fetch_add(1);
    return SEGATTN_OK;
}

// Forward over a prepared head table (shared by seg_attn_fwd and the streamed prefill).
segattn_status launch_fwd(const seg_attn_params* p, const HeadTable& heads, const void* Q, const void* K,
                          const void* V, void* O, float* LSE, cudaStream_t stream) {
    if (p->B == 0 || p->Lq == 0 || heads.n_slots == 0) return SEGATTN_OK;
    FwdParams prm;
    memset(&prm, 0, sizeof(prm));
    segattn_status st;
    const void* kbase = p->kv_len > 0 ? K : Q;  // kv_len == 0: maps are never dereferenced
    const void* vbase = p->kv_len > 0 ? V : Q;
    if ((st = make_map(&prm.tq, Q, p->d, p->Hq, p->Lq, p->B, p->q_stride)) != SEGATTN_OK) return st;
    if ((st = make_map(&prm.tk, kbase, p->d, heads.n_slots, p->kv_len, p->B, p->kv_len > 0 ? p->k_stride : p->q_stride)) !=
        SEGATTN_OK)
        return st;
    if ((st = make_map(&prm.tv, vbase, p->d, heads.n_slots, p->kv_len, p->B, p->kv_len > 0 ? p->v_stride : p->q_stride)) !=
        SEGATTN_OK)
        return st;
    if ((st = make_map(&prm.to, O, p->d, p->Hq, p->Lq, p->B, p->o_stride)) != SEGATTN_OK) return st;
    prm.O = O;
    prm.LSE = LSE;
    for (int i = 0; i < 3; ++i) prm.o_stride[i] = p->o_stride[i];
    prm.geom = geom_of(p);
    prm.B = p->B;
    prm.Hq = p->Hq;
    prm.g = p->Hq / p->Hkv;
    prm.n_qtiles = (p->Lq + kTile - 1) / kTile;
    prm.scale_log2 = p->sm_scale * 1.4426950408889634f;
    prm.heads = heads;
    const long long n_items = (long long)p->B * heads.n_slots * prm.g * prm.n_qtiles;
    if (n_items > 0x7fffffffLL) return SEGATTN_ERR_INVALID;
    prm.n_items = (int)n_items;
    set_decode_divisors(prm, heads, prm.g, p->B);
    // persistent: one CTA per SM walks the work list
    int n_sm = 0;
    if ((st = sm_count(&n_sm)) != SEGATTN_OK) return st;
    const unsigned grid = (unsigned)(n_items < n_sm ? n_items : n_sm);
    if (log_on())
        fprintf(stderr, "[segattn] fwd: B=%d Lq=%d kv_len=%d Hq=%d Hkv=%d d=%d S=%d T=%d q_pos0=%d kv_pos0=%d segs=%d "
                        "slots=%d past_slots=%d items=%lld grid=%u\n",
                p->B, p->Lq, p->kv_len, p->Hq, p->Hkv, p->d, p->S, p->T, p->q_pos0, p->kv_pos0, prm.geom.n_starts,
                heads.n_slots, heads.n_flagged, n_items, grid);
    if (p->d == 128) {
        if ((st = set_smem(seg_attn_fwd_kernel<128>, FwdSmem<128>::kDynamic)) != SEGATTN_OK) return st;
        seg_attn_fwd_kernel<128><<<grid, kFwdThreads, FwdSmem<128>::kDynamic, stream>>>(prm);
    } else {
        if ((st = set_smem(seg_attn_fwd_kernel<64>, FwdSmem<64>::kDynamic)) != SEGATTN_OK) return st;
        seg_attn_fwd_kernel<64><<<grid, kFwdThreads, FwdSmem<64>::kDynamic, stream>>>(prm);
    }
    return launch_check();
}

size_t round256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace

extern "C" {

size_t seg_attn_workspace_bytes(const seg_attn_params* p, int is_bwd) {
    if (!params_ok(p)) return 0;
    if (!is_bwd) return 0;
    return round256((size_t)p->B * p->Hq * p->Lq * sizeof(float));
}

segattn_status seg_attn_fwd(const seg_attn_params* p, const void* Q, const void* K, const void* V,
                            const uint8_t* head_past_mask, void* O, float* LSE, void* workspace,
                            size_t workspace_bytes, void* stream) {
    (void)workspace;
    (void)workspace_bytes;
    if (!params_ok(p) || !mask_ok(head_past_mask, p->Hkv)) return SEGATTN_ERR_INVALID;
    if (!strides_ok(p->q_stride, p->d) || !strides_ok(p->k_stride, p->d) || !strides_ok(p->v_stride, p->d) ||
        !strides_ok(p->o_stride, p->d))
        return SEGATTN_ERR_INVALID;
    if (p->B > 0 && p->Lq > 0) {
        if (!Q || !O || !LSE || !aligned16(Q) || !aligned16(O) || (reinterpret_cast<uintptr_t>(LSE) & 3u))
            return SEGATTN_ERR_INVALID;
        if (p->kv_len > 0 && (!K || !V || !aligned16(K) || !aligned16(V))) return SEGATTN_ERR_INVALID;
    }
    segattn_status st = check_arch();
    if (st != SEGATTN_OK) return st;
    HeadTable heads;
    identity_heads(&heads, p->Hkv, head_past_mask);
    return launch_fwd(p, heads, Q, K, V, O, LSE, static_cast<cudaStream_t>(stream));
}

segattn_status seg_attn_poll_status(void* stream) {
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    int word = 0;
    e = cudaMemcpyFromSymbol(&word, g_device_status, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
    if (word == 0) return SEGATTN_OK;
    t_last_cuda_error = word;
    int zero = 0;
    e = cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
    // the word is (status << 8) | detail: an expired wait, or input a kernel refused (an index out of range)
    return (word >> 8) == SEGATTN_ERR_INVALID ? SEGATTN_ERR_INVALID : SEGATTN_ERR_TIMEOUT;
}

const char* seg_attn_status_string(segattn_status s) {
    switch (s) {
        case SEGATTN_OK: return "ok";
        case SEGATTN_ERR_INVALID: return "invalid argument";
        case SEGATTN_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x (B200)";
        case SEGATTN_ERR_CUDA: return "CUDA call failed";
        case SEGATTN_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
        case SEGATTN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SEGATTN_ERR_TOO_LARGE:
            return "problem exceeds the fixed scratch of seg_attn_bwd_static (B*Hq*Lq > SEG_ATTN_STATIC_MAX_ROWS)";
    }
    return "unknown status";
}

int seg_attn_last_cuda_error(void) { return t_last_cuda_error; }

int64_t seg_attn_launch_count(void) { return g_launches.load(); }

segattn_status seg_attn_count_pairs(const seg_attn_params* p, const uint8_t* head_past_mask, int64_t* pairs_visible,
                                    int64_t* pairs_diff, int64_t* fwd_tiles) {
    if (!params_ok(p) || !mask_ok(head_past_mask, p->Hkv)) return SEGATTN_ERR_INVALID;
    const MaskGeom g = geom_of(p);
    const int grp = p->Hq / p->Hkv;
    long long vis = 0, dif = 0, tiles = 0;
    for (int c = 0; c < p->Hkv; ++c) {
        const int f = head_past_mask[c];
        long long v = 0, d = 0, t = 0;
        for (int r = 0; r < p->Lq; ++r) {
            const long long pos = (long long)g.q_pos0 + r;
            long long hi = pos - g.kv_pos0;
            if (hi > g.kv_len - 1) hi = g.kv_len - 1;
            long long lo = lo_visible(g, pos, f) - g.kv_pos0, lod = lo_diff(g, pos, f) - g.kv_pos0;
            if (lo < 0) lo = 0;
            if (lod < 0) lod = 0;
            if (hi >= lo) v += hi - lo + 1;
            if (hi >= lod) d += hi - lod + 1;
        }
        for (int r0 = 0; r0 < p->Lq; r0 += kTile) {
            long long a, b;
            q_tile_kv_range(g, r0, f, false, &a, &b);
            if (b >= a) t += b / kTile - a / kTile + 1;
        }
        vis += v * grp;
        dif += d * grp;
        tiles += t * grp;
    }
    if (pairs_visible) *pairs_visible = vis * p->B;
    if (pairs_diff) *pairs_diff = dif * p->B;
    if (fwd_tiles) *fwd_tiles = tiles * p->B;
    return SEGATTN_OK;
}

}  // extern "C"

#include "seg_attn_bwd_api.inc"
#include "seg_attn_prefill_api.inc"
#include "seg_attn_rope_api.inc"

// ---- Self-test of the bounded waits ------------------------------------------------------------
namespace {
// One warp waits on an mbarrier nobody arrives on, with a 1 ms limit: the wait gives up, records
// site 99 in the status word and the kernel returns normally.
__global__ void selftest_wait_kernel() {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) mbar_wait_slow(smem_u32(&bar), 0, 99, 1000000ull);
}
}  // namespace

extern "C" segattn_status seg_attn_selftest_wait_timeout(void* stream) {
    segattn_status st = check_arch();
    if (st != SEGATTN_OK) return st;
    selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>();
    return launch_check();
}

// ---- Backward without a caller-provided workspace ---------------------------------------------
// The row dots D = <dO, O> of seg_attn_bwd_static live here instead of in caller memory.  In host
// code this name is only a handle for the runtime's symbol calls, never a device address: the
// address the kernels get comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) float g_static_row_dots[SEG_ATTN_STATIC_MAX_ROWS];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
float* g_static_ptr[kMaxDevices] = {};  // per device: address of g_static_row_dots on that device

// Device address of the static scratch on the current device (first use per device: one symbol look-up).
segattn_status static_scratch(float** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return SEGATTN_ERR_INVALID;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_row_dots);
        if (e != cudaSuccess) return cuda_fail(e);
        if (!ptr) return SEGATTN_ERR_CUDA;
        g_static_ptr[dev] = static_cast<float*>(ptr);
    }
    *out = g_static_ptr[dev];
    return SEGATTN_OK;
}

}  // namespace

extern "C" segattn_status seg_attn_bwd_static(const seg_attn_params* p, const void* Q, const void* K, const void* V,
                                              const void* O, const float* LSE, const void* dO,
                                              const uint8_t* head_past_mask, void* dQ, void* dK, void* dV,
                                              void* stream) {
    if (!params_ok(p) || !mask_ok(head_past_mask, p->Hkv) || !all_strides_ok(p)) return SEGATTN_ERR_INVALID;
    const bool have_q = p->B > 0 && p->Lq > 0, have_kv = p->B > 0 && p->kv_len > 0;
    if (have_q && (!Q || !O || !LSE || !dO || !dQ || !aligned16(Q) || !aligned16(O) || !aligned16(dO) || !aligned16(dQ) ||
                   (reinterpret_cast<uintptr_t>(LSE) & 3u)))
        return SEGATTN_ERR_INVALID;
    if (have_kv && (!K || !V || !dK || !dV || !aligned16(K) || !aligned16(V) || !aligned16(dK) || !aligned16(dV)))
        return SEGATTN_ERR_INVALID;
    if ((long long)p->B * p->Hq * p->Lq > (long long)SEG_ATTN_STATIC_MAX_ROWS) return SEGATTN_ERR_TOO_LARGE;
    segattn_status st = check_arch();
    if (st != SEGATTN_OK) return st;
    float* row_dots = nullptr;
    if ((st = static_scratch(&row_dots)) != SEGATTN_OK) return st;
    HeadTable heads;
    identity_heads(&heads, p->Hkv, head_past_mask);
    return launch_bwd(p, heads, Q, K, V, O, LSE, dO, dQ, dK, dV, row_dots, static_cast<cudaStream_t>(stream));
}

#ifdef SEGATTN_TRACE
// Debug builds only: choose the traced CTA / read back its clock stamps.
extern "C" int seg_attn_debug_trace(long long* out, int n, int set_block) {
    if (set_block >= 0) {
        static long long zeros[4096];
        const int kernel_id = set_block >> 24;  // 0 forward, 1 dQ pass, 2 dK/dV pass
        set_block &= 0xffffff;
        cudaMemcpyToSymbol(g_trace_kernel, &kernel_id, sizeof(int));
        cudaMemcpyToSymbol(g_trace_block, &set_block, sizeof(int));
        cudaMemcpyToSymbol(g_trace, zeros, sizeof(zeros));
        return 0;
    }
    cudaDeviceSynchronize();
    return (int)cudaMemcpyFromSymbol(out, g_trace, sizeof(long long) * (n < 4096 ? n : 4096));
}
#endif

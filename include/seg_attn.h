/*
 * seg_attn.h - C ABI of the segment-level causal attention library for NVIDIA B200 (sm_100a).
 *
 * The operation (names follow the paper; its total length T is `L` here, its tail length M is `T`):
 * a sequence of L positions is cut into non-overlapping segments of constant length S
 * (Section 3.1 "Setup", Section 3.5).  Every head runs scaled dot-product attention
 * softmax(Q K^T * sm_scale + mask) V (Appendix C, Eq. "attn") over a per-segment context
 * (Appendix C, Eq. "ctx"):
 *   - its own segment, causally (a query sees positions up to and including itself);
 *   - the carried KV tail: the last T key/value positions of the immediately preceding
 *     segment, the only differentiable cross-segment state (Section 3.4, "Local Continuity
 *     Channel"); the first segment has no carried state (Section 3.1, C_0 empty);
 *   - for KV heads of class SEGATTN_HEAD_PAST in `head_past_mask`, additionally every older
 *     key/value, read forward-only: stop-gradient, no gradient reaches those K/V (Definition 3.2;
 *     Section 3.4, "Long-Range Channel"; Appendix B, Lemma B.1);
 *   - KV heads of class SEGATTN_HEAD_OWN read their own segment and nothing else: the context of
 *     a long-range head in a layer that is not a long-range layer (Appendix C, Eq. "ctx", third
 *     case).
 * With global positions p (query) and j (key), i = p / S and a_i = max(0, i*S - T):
 *     visible(p, j, c) <=> lo_c(p) <= j <= p,  lo_c(p) = a_i (LOCAL), 0 (PAST), i*S (OWN)
 *     diff(p, j, c)    <=> max(lo_c(p), a_i) <= j <= p   (reads that carry gradient into K/V)
 * With seg_attn_params.seg_starts the segments have the lengths the caller gives instead of S: i is the
 * segment that holds p, i*S becomes its start s_i, and a_i = max(s_{i-1}, s_i - T) (the carried tail of a
 * segment shorter than T is the whole segment).
 * Query head h uses KV head c = h / (Hq / Hkv).
 *
 * Conventions that hold for every entry point unless it says otherwise:
 *   - Tensor pointers are DEVICE pointers owned by the caller; the library never frees or
 *     reallocates them.  Q, O, dO, dQ are bf16 [B][Lq][Hq][d]; K, V, dK, dV are bf16
 *     [B][kv_len][Hkv][d]; addressing is by the element strides in seg_attn_params (the last
 *     dimension is contiguous).  LSE is fp32, contiguous [B][Hq][Lq].
 *   - `head_past_mask` is a HOST array of Hkv bytes, one head class per KV head (0 = local,
 *     1 = past access, 2 = own segment only; any other value is SEGATTN_ERR_INVALID); it is read
 *     before the call returns.
 *   - `stream` is a cudaStream_t passed as void*.  Work is enqueued on it; no entry point
 *     synchronises the device except where stated.
 *   - Errors are return codes.  Arguments are validated on the host before anything is
 *     launched: SEGATTN_ERR_INVALID, _UNSUPPORTED_ARCH, _WORKSPACE and _TOO_LARGE mean that nothing
 *     was enqueued and the outputs are untouched.  SEGATTN_ERR_CUDA can also come from a launch or
 *     copy in the middle of a call's sequence (a backward is three kernels, the host-buffer step
 *     and the streamed prefill several launches and copies): what was enqueued before it still
 *     runs, so treat the outputs, and for the streamed prefill the handle's state, as undefined.
 *   - The kernels share one device status word per process (see seg_attn_poll_status).  Once a
 *     kernel has set it - a bounded wait that ran out, an index a kernel refused - later kernels
 *     give up their waits early too, so outputs enqueued after that are undefined until
 *     seg_attn_poll_status has been called, which reads and clears the word.
 *   - Base pointers must be 16-byte aligned and every stride a multiple of 8 elements
 *     (tiles are moved by TMA).  d is 64 or 128.  0 <= T <= S.  Any Lq, kv_len >= 0.
 *   - Arithmetic: bf16 inputs, fp32 accumulation on the tensor cores, fp32 softmax
 *     statistics; P (and dS) are rounded to bf16 before the second product; outputs are
 *     rounded to bf16 (round-to-nearest-even).  A query row with no visible key present
 *     (possible only when kv_len does not reach it) yields O = 0, LSE = -inf.
 */
#ifndef SEG_ATTN_H_
#define SEG_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SEGATTN_OK = 0,
    SEGATTN_ERR_INVALID = 1,          /* bad shape, stride, alignment, null pointer, T > S, unsupported d */
    SEGATTN_ERR_UNSUPPORTED_ARCH = 2, /* the current device is not compute capability 10.x */
    SEGATTN_ERR_CUDA = 3,             /* a CUDA runtime/driver call failed; see seg_attn_last_cuda_error() */
    SEGATTN_ERR_TIMEOUT = 4,          /* a bounded wait inside a kernel expired (see seg_attn_poll_status) */
    SEGATTN_ERR_WORKSPACE = 5,        /* workspace/state buffer missing, misaligned or too small */
    SEGATTN_ERR_TOO_LARGE = 6         /* problem exceeds the fixed scratch of seg_attn_bwd_static */
} segattn_status;

/* Head classes, the entries of `head_past_mask` (Appendix C, Eq. "ctx"). */
#define SEGATTN_HEAD_LOCAL 0 /* own segment + carried tail, both differentiable */
#define SEGATTN_HEAD_PAST 1  /* own segment + carried tail + every older position (forward-only) */
#define SEGATTN_HEAD_OWN 2   /* own segment only */

/* seg_attn_params.flags, bit 0: for flagged KV heads the reads of the carried tail are stop-gradient
 * too, i.e. diff(p, j) <=> i*S <= j <= p for them.  This is the literal reading of Appendix C,
 * Eq. "ctx", where only local heads build and read the differentiable carried state and long-range
 * heads see their prefix forward-only.  The forward is the same in both readings; only the set of
 * (query, key) pairs that feed dK/dV changes. */
#define SEGATTN_FLAG_FLAGGED_TAIL_SG 1

typedef struct {
    int32_t B;       /* batch */
    int32_t Lq;      /* number of query rows per batch element */
    int32_t kv_len;  /* number of key/value rows present per batch element */
    int32_t Hq;      /* query heads */
    int32_t Hkv;     /* key/value heads; Hq % Hkv == 0; at most 64 */
    int32_t d;       /* head dimension: 64 or 128 */
    int32_t S;       /* segment length, >= 1 */
    int32_t T;       /* carried tail length, 0 <= T <= S */
    int32_t q_pos0;  /* global position of query row 0 (0 for a whole sequence; i*S when streaming) */
    int32_t kv_pos0; /* global position of key row 0 (may be negative: rows before position 0 are never visible) */
    float sm_scale;  /* softmax scale; the paper uses 1/sqrt(d) */
    int32_t flags;   /* bit set of SEGATTN_FLAG_*; 0 for the default semantics */
    int32_t detach_before; /* backward only: keys at global positions below this are read forward-only
                            * (no dK/dV from them, and their dK/dV rows come out zero): the boundary
                            * state of a truncated chain enters as a constant (K-truncated objective,
                            * Eq. "truncated-base").  A window of K+1 segments passes the position of
                            * its first segment.  0: none.  Must be >= 0. */
    int64_t q_stride[3]; /* element strides of Q (and dQ) for (batch, position, head) */
    int64_t k_stride[3]; /* element strides of K (and dK) */
    int64_t v_stride[3]; /* element strides of V (and dV) */
    int64_t o_stride[3]; /* element strides of O (and dO) */
    const int32_t* seg_starts; /* NULL: segments of constant length S.  Else a HOST array of n_segs ascending global
                                * positions, the first 0: segment i is [seg_starts[i], seg_starts[i+1]) and the last one
                                * is open-ended (segments of lengths m_i, Section 3.1).  S is then ignored, T may exceed
                                * a segment's length (the carried tail of a short segment is the whole segment).  The
                                * streamed prefill driver takes its lengths step by step instead (seg_prefill_step_len).  Read before the call returns. */
    int32_t n_segs;            /* 1 .. 256 when seg_starts is given */
} seg_attn_params;

/* Bytes of device scratch a call needs (is_bwd = 0: forward, none today; 1: backward, the
 * fp32 row dots D[B][Hq][Lq], rounded up to 256).  Returns 0 for invalid params. */
size_t seg_attn_workspace_bytes(const seg_attn_params* p, int is_bwd);

/* Forward (Appendix C, Eqs. "attn" and "ctx"; mask as stated at the top of this file).
 * O[b][r][h][:] = sum_j P_j V_j and LSE[b][h][r] = ln sum_j exp(sm_scale * <q,k_j>) over the
 * visible j (natural logarithm of the scaled scores).  Fully overwrites O and LSE.
 * `workspace` may be NULL (size 0). */
segattn_status seg_attn_fwd(const seg_attn_params* p, const void* Q, const void* K, const void* V,
                            const uint8_t* head_past_mask, void* O, float* LSE,
                            void* workspace, size_t workspace_bytes, void* stream);

/* Backward: the vector-Jacobian product of the forward for the cotangent dO (softmax VJP;
 * stop-gradient per Definition 3.2 and Lemma B.1; the tail as sole differentiable
 * cross-segment state per Section 3.4; one-transition reach of the K=1 discussion after
 * Definition 3.2).  With P = exp(s - LSE), D = <dO,O>, dS = P * (dO V^T - D):
 *   dQ_p = sm_scale * sum over visible j of dS_pj K_j          (stop-gradient keys included:
 *                                                               sg cuts the K/V side only)
 *   dK_j = sm_scale * sum over p with diff(p,j) of dS_pj Q_p,  dV_j = sum over the same p of P_pj dO_p
 * summed over the query heads of the KV head.  A key position thus receives gradient only
 * from queries of its own segment and, if it lies in the last T positions, of the next one.
 * O and LSE must be the forward's results for the same inputs.  dQ, dK, dV are fully
 * overwritten (no pre-zeroing).  `workspace` must hold seg_attn_workspace_bytes(p, 1) bytes,
 * 256-byte aligned; it is scratch, dead after the enqueued work has run. */
segattn_status seg_attn_bwd(const seg_attn_params* p, const void* Q, const void* K, const void* V,
                            const void* O, const float* LSE, const void* dO,
                            const uint8_t* head_past_mask, void* dQ, void* dK, void* dV,
                            void* workspace, size_t workspace_bytes, void* stream);

/* Backward for callers that cannot allocate device memory (the paper has no counterpart; this is
 * a packaging variant of seg_attn_bwd, not another operation).  Some hosts of this library may
 * not call cudaMalloc where the backward runs - a serving or training loop whose memory pool is
 * sized at start-up and frozen, a plugin that is handed tensors but no allocator, code that must
 * not trigger the implicit device synchronisation an allocation can cause - and so cannot provide
 * the `workspace` seg_attn_bwd asks for.  This entry point takes
 * no workspace: the fp32 row dots D live in a fixed array inside the library's device image,
 * SEG_ATTN_STATIC_MAX_ROWS floats (4 MiB) that every GPU loading the library holds until the
 * process exits.  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - Same arguments, results and error codes as seg_attn_bwd otherwise (same kernels).
 *   - Problems with B * Hq * Lq > SEG_ATTN_STATIC_MAX_ROWS are rejected with
 *     SEGATTN_ERR_TOO_LARGE before anything is launched; use seg_attn_bwd with a workspace.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress, with that device current).  Make that first call outside any stream
 *     capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents (every
 *     element a call reads it has written first, so nothing needs clearing).  Two calls whose
 *     work overlaps on the GPU - different streams, or threads - race on it: serialise them. */
#define SEG_ATTN_STATIC_MAX_ROWS (1 << 20)
segattn_status seg_attn_bwd_static(const seg_attn_params* p, const void* Q, const void* K, const void* V,
                                   const void* O, const float* LSE, const void* dO,
                                   const uint8_t* head_past_mask, void* dQ, void* dK, void* dV, void* stream);

/* ---- Streamed prefill: the segment recurrence (C_i, o_i) = F(x_i, C_{i-1}, R_{i-1}) of
 * Definition 3.1 restricted to attention, with memory bounded as in Section 3.5 "Memory
 * Complexity": flagged KV heads keep their whole key/value history (the append-only
 * past-only pool of Section 3.4), the others keep only the T-position tail.
 *
 * The caller provides one device buffer for all persistent state.  In `p`, Lq is the
 * segment length fed per step (must equal S; seg_prefill_step_len feeds shorter ones), kv_len is the
 * maximum total length the pool must hold, q_pos0/kv_pos0 are ignored, and the Q/O strides describe the per-step
 * Q/O segment tensors [B][S][Hq][d], the K/V strides the per-step K/V segment tensors
 * [B][S][Hkv][d].  The handle itself is a small host object (malloc'd by create, freed by
 * destroy). */
typedef struct seg_prefill_handle seg_prefill_handle;

size_t seg_prefill_state_bytes(const seg_attn_params* p, const uint8_t* head_past_mask);
segattn_status seg_prefill_create(const seg_attn_params* p, const uint8_t* head_past_mask,
                                  void* state_mem, size_t state_bytes, seg_prefill_handle** out);
/* Processes the next segment: appends its K/V to the retained state, writes O_seg
 * [B][S][Hq][d] and LSE_seg [B][Hq][S] (the same values the whole-sequence forward gives for
 * those rows), then rolls the tail.  Call once per segment, in order, on one stream. */
segattn_status seg_prefill_step(seg_prefill_handle* h, const void* Qseg, const void* Kseg, const void* Vseg,
                                void* Oseg, float* LSEseg, void* stream);
/* The same for a segment of Lseg rows, 1 <= Lseg <= S: segments of lengths m_i (Section 3.1 lets them differ), and
 * in particular a shorter last segment.  The segment tensors hold Lseg rows per batch element and are addressed with
 * the strides given at creation; LSE_seg is [B][Hq][Lseg].  The carried tail of a segment shorter than T is the whole
 * segment (never more than one segment back), as with seg_attn_params.seg_starts, whose whole-sequence forward this
 * reproduces row for row.  seg_prefill_step(h, ...) is seg_prefill_step_len(h, S, ...). */
segattn_status seg_prefill_step_len(seg_prefill_handle* h, int32_t Lseg, const void* Qseg, const void* Kseg,
                                    const void* Vseg, void* Oseg, float* LSEseg, void* stream);
/* Backward of the segment stepped last (the streamed form of training with truncation depth 1: a
 * segment is run forward, its loss is differentiated, and credit stops where the carried state
 * entered - definition of the K-truncated objective with K = 1).  Valid after seg_prefill_step and
 * before the next one; the state still holds what that step attended over.  Qseg, Oseg, dOseg and
 * dQseg hold the Lseg rows of that step per batch element ([B][S][Hq][d] for a full segment) with the strides
 * given at creation, LSEseg as returned by the step.
 * dKctx and dVctx are contiguous bf16 [B][T+S][Hkv][d]: the gradients of the key/value rows at
 * global positions [pos - T, pos + Lseg), pos the segment's start - the T positions in front of the segment, of
 * which the previous segment's carried tail (its last min(T, length) positions) can be non-zero, then the segment
 * itself; rows before position 0 and the S - Lseg rows after a shorter segment are zero.  Older rows of past-access
 * heads are read forward-only and get none.  The caller adds the first T rows to the previous segment's gradients.  `workspace`: DEVICE,
 * 256-byte aligned, at least seg_prefill_bwd_workspace_bytes(h) bytes.  SEGATTN_ERR_INVALID when no segment
 * has been stepped yet or a pointer is null or misaligned, SEGATTN_ERR_WORKSPACE for the workspace; the state
 * is not modified. */
size_t seg_prefill_bwd_workspace_bytes(const seg_prefill_handle* h);
segattn_status seg_prefill_step_bwd(seg_prefill_handle* h, const void* Qseg, const void* Oseg, const float* LSEseg,
                                    const void* dOseg, void* dQseg, void* dKctx, void* dVctx, void* workspace,
                                    size_t workspace_bytes, void* stream);
segattn_status seg_prefill_reset(seg_prefill_handle* h); /* back to segment 0; state contents become dead */
void seg_prefill_destroy(seg_prefill_handle* h);

/* ---- Context of a head that reads a retrieved prefix (Appendix C, Eq. "ctx", first case: a
 * long-range head in a long-range layer attends over [K_ret ; K_i], R retrieved rows followed by
 * its own segment; Appendix D fixes R positions per head).  Given the R positions, builds
 *     K_ctx[b][r][c][:]     = K_pool[b][idx[b][c][r]][c][:]      0 <= r < R
 *     K_ctx[b][R + t][c][:] = K_seg[b][t][c][:]                  0 <= t < Lseg
 * and V_ctx alike.  K_pool/V_pool are bf16 with element strides pool_stride (batch, position, head)
 * and pool_len positions; K_seg/V_seg likewise with seg_stride; K_ctx/V_ctx are contiguous
 * [B][R + Lseg][Hkv][d].  idx is a DEVICE array of int32, [B][Hkv][R].  All pointers 16-byte
 * aligned, strides multiples of 8.  An index outside [0, pool_len) is not read: its row is zero
 * and the next seg_attn_poll_status returns SEGATTN_ERR_INVALID.  The attention itself is the
 * existing entry points on the context: seg_attn_fwd / seg_attn_bwd with Lq = Lseg, kv_len = R + Lseg,
 * q_pos0 = R, kv_pos0 = 0, S = R + Lseg, T = 0, class 0 heads, and, in the backward,
 * detach_before = R (the retrieved rows are forward-only: Definition 3.2, Lemma B.1); rows
 * [R, R + Lseg) of the dK/dV it returns are the segment's gradients.  The R positions come from the
 * caller or from seg_retrieval_select below. */
segattn_status seg_attn_gather_context(int32_t B, int32_t Hkv, int32_t d, int32_t R, int32_t Lseg, int32_t pool_len,
                                       const void* K_pool, const void* V_pool, const int64_t pool_stride[3],
                                       const void* K_seg, const void* V_seg, const int64_t seg_stride[3],
                                       const int32_t* idx, void* K_ctx, void* V_ctx, void* stream);

/* ---- Selection step of the top-k retrieval operator (Appendix D): which R pool positions a head
 * retrieves.  The paper names the steps and states none of the constants, so all are parameters here,
 * and the tie and overflow rules are this library's (equal scores: lower position first; windows are
 * added best anchor first until R positions are chosen; a short set is padded with the earliest
 * positions not yet chosen).  Steps per (batch, KV head): (1) query summaries of the last Lq_last
 * queries of the previous segment - the mean over each sliding window [u*stride, u*stride + window)
 * and the mean over the last `tail` rows, averaged over the group's query heads; (2) dot-product
 * scores of every summary against every pool key; (3) the top_k keys per summary, deduplicated;
 * (4) the n_anchors candidates of highest score; (5) positions anchor - off_lo .. anchor + off_hi,
 * padded to exactly R, ascending.  Arithmetic is fp32 with separately rounded products and
 * sequential sums, so the choice is reproducible bit for bit.  Q_last is bf16, contiguous
 * [B][Lq_last][Hq][d]; K_pool bf16 with element strides pool_stride (batch, position, head) and P
 * positions; idx (DEVICE, int32 [B][Hkv][R]) is what seg_attn_gather_context takes.  Limits: at most
 * 16 summaries, summaries * top_k <= 1024, R <= P, top_k <= P.  `workspace`: DEVICE, 256-byte aligned,
 * seg_retrieval_workspace_bytes(...) bytes (0 = invalid parameters).  Returns SEGATTN_ERR_INVALID for
 * parameters outside these limits or misaligned pointers and SEGATTN_ERR_WORKSPACE for a missing, misaligned
 * or short workspace, before anything is launched; the workspace's contents are scratch. */
typedef struct {
    int32_t Lq_last, window, stride, tail; /* query summaries */
    int32_t top_k, n_anchors;              /* candidates per summary; anchors kept */
    int32_t off_lo, off_hi;                /* window around an anchor */
    int32_t R;                             /* positions returned per head */
} seg_retrieval_params;
size_t seg_retrieval_workspace_bytes(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t P, const seg_retrieval_params* r);
segattn_status seg_retrieval_select(int32_t B, int32_t Hq, int32_t Hkv, int32_t d, int32_t P, const void* Q_last,
                                    const void* K_pool, const int64_t pool_stride[3], const seg_retrieval_params* r,
                                    int32_t* idx, void* workspace, size_t workspace_bytes, void* stream);

/* ---- RoPE re-indexing for prefix concatenation (Section 3.4, paragraph of that name; Appendix E).  When a
 * prefix of P key/value rows - the carried tail (P = T) or the retrieved rows (P = R) - is put in front of a
 * segment of m rows, the prefix keys are rotated with positions 0 .. P-1 and the segment's queries and keys with
 * positions P .. P+m-1; values are not rotated.  (For the carried tail this equals rotating everything at its
 * global position, since scores depend on position differences only; for retrieved rows it does not, which is
 * why the pool must hold keys BEFORE rotation.)  "Standard RoPE" is read as the rotation of the pairs
 * (x[i], x[i + d/2]), i < d/2, by the angle pos * base^(-2i/d):
 *     y[i] = x[i] cos a - x[i + d/2] sin a,   y[i + d/2] = x[i] sin a + x[i + d/2] cos a.
 * The angles' cosines and sines come from a table the caller keeps on the device:
 *   seg_rope_table_bytes   bytes of a table for positions [0, n_pos) (0: invalid d or n_pos; n_pos <= 2^24);
 *   seg_rope_table         fills `table` (DEVICE, 16-byte aligned, fp32 [n_pos][d/2][2] = (cos, sin)); the angles are
 *                          formed and their cosines and sines taken in double precision, then rounded to fp32;
 *   seg_rope_apply         Y[b][r][h][:] = Rot(pos0 + r) X[b][r][h][:] for bf16 X, Y [B][L][H][d] with the element
 *                          strides given (batch, row, head; multiples of 8; Y may be X); inverse != 0 applies the
 *                          transposed rotation, which maps a gradient with respect to the rotated tensor back to one
 *                          with respect to the unrotated tensor (dQ of the segment, and rows [R, R+m) of dK).
 *                          Arithmetic fp32, output rounded to bf16.  pos0 + L <= n_pos.
 *   seg_attn_gather_context_rope   seg_attn_gather_context with the re-indexed rotation applied to the keys while
 *                          they are copied: K_ctx[b][r][c] = Rot(r) K_pool[b][idx[b][c][r]][c] for r < R,
 *                          K_ctx[b][R + t][c] = Rot(R + t) K_seg[b][t][c]; V_ctx is the plain copy.  Same arguments,
 *                          limits and error behaviour as seg_attn_gather_context; R + Lseg <= n_pos.  The segment's
 *                          queries are rotated by seg_rope_apply with pos0 = R.
 * All four validate their arguments on the host (SEGATTN_ERR_INVALID) and enqueue one kernel on `stream`. */
size_t seg_rope_table_bytes(int32_t n_pos, int32_t d);
segattn_status seg_rope_table(int32_t n_pos, int32_t d, double base, float* table, void* stream);
segattn_status seg_rope_apply(int32_t B, int32_t L, int32_t H, int32_t d, const void* X, const int64_t x_stride[3],
                              void* Y, const int64_t y_stride[3], int32_t pos0, int32_t inverse, const float* table,
                              int32_t n_pos, void* stream);
segattn_status seg_attn_gather_context_rope(int32_t B, int32_t Hkv, int32_t d, int32_t R, int32_t Lseg, int32_t pool_len,
                                            const void* K_pool, const void* V_pool, const int64_t pool_stride[3],
                                            const void* K_seg, const void* V_seg, const int64_t seg_stride[3],
                                            const int32_t* idx, void* K_ctx, void* V_ctx, const float* table,
                                            int32_t n_pos, void* stream);

/* ---- Whole training-step call with HOST buffers (pinned or pageable): copies Q, K, V, dO to
 * the device arena, runs forward and backward, copies O, LSE, dQ, dK, dV back, and
 * synchronises `stream` before returning.  Host tensors are contiguous in the layouts
 * above (strides in `p` are ignored).  dO_host == NULL runs the forward only (gradient
 * outputs are then ignored).  `arena` is a caller-owned DEVICE buffer of at least
 * seg_attn_host_arena_bytes(p) bytes, 256-byte aligned.  The work is processed in up to eight
 * chunks - ranges of batch elements or, for batches smaller than that, ranges of KV heads (with
 * their query heads) of one batch element, each an independent problem - whose copies in, kernels
 * (on `stream`) and copies out overlap; the two side streams and their events are created on first
 * use per device and kept for the life of the process.
 * With pageable host memory the copies do not overlap but the result is the same. */
size_t seg_attn_host_arena_bytes(const seg_attn_params* p);
segattn_status seg_attn_step_host(const seg_attn_params* p, const void* Q_host, const void* K_host,
                                  const void* V_host, const void* dO_host, const uint8_t* head_past_mask,
                                  void* O_host, float* LSE_host, void* dQ_host, void* dK_host, void* dV_host,
                                  void* arena, size_t arena_bytes, void* stream);

/* ---- Status and accounting */
/* Synchronises `stream`, then reads and clears the device status word that kernels set when a
 * bounded wait expires or a kernel refuses its input.  Returns SEGATTN_OK, SEGATTN_ERR_TIMEOUT,
 * SEGATTN_ERR_INVALID (an index out of range in seg_attn_gather_context) or SEGATTN_ERR_CUDA. */
segattn_status seg_attn_poll_status(void* stream);
const char* seg_attn_status_string(segattn_status s);
/* Last CUDA error code (cudaError_t or CUresult as int) recorded by this thread's failing call. */
int seg_attn_last_cuda_error(void);
/* Exact (query,key) pair counts of the mask summed over batch and query heads (the cost
 * model of Section 3.5 evaluated element-exactly), and the number of 128x128 tiles the
 * forward kernel visits.  Any of the output pointers may be NULL. */
segattn_status seg_attn_count_pairs(const seg_attn_params* p, const uint8_t* head_past_mask,
                                    int64_t* pairs_visible, int64_t* pairs_diff, int64_t* fwd_tiles);
/* Measurement aid (the paper has no counterpart): runs each of the four kernels of a training
 * step on its own - forward, row dots, dQ pass, dK/dV pass, in that order - once untimed and then
 * `iters` times back to back between two CUDA events recorded on `stream`, and returns the average
 * milliseconds per launch in ms_per_launch[0..3].  Arguments as for seg_attn_fwd / seg_attn_bwd
 * (O and LSE are written by the forward and read by the backward).  Synchronises `stream`. */
segattn_status seg_attn_profile_kernels(const seg_attn_params* p, const void* Q, const void* K, const void* V,
                                       void* O, float* LSE, const void* dO, const uint8_t* head_past_mask, void* dQ,
                                       void* dK, void* dV, void* workspace, size_t workspace_bytes, int iters,
                                       float ms_per_launch[4], void* stream);
/* Diagnostic aid (the paper has no counterpart): enqueues a one-warp kernel that waits, with a
 * 1 ms limit, on a barrier nothing ever signals - the way every wait inside the library's kernels
 * is bounded.  The wait gives up, the kernel ends normally, and the next seg_attn_poll_status
 * returns SEGATTN_ERR_TIMEOUT (seg_attn_last_cuda_error() then gives (4 << 8) | 99) and clears
 * the status word; the context stays usable. */
segattn_status seg_attn_selftest_wait_timeout(void* stream);
/* Number of kernel launches the library has enqueued so far in this process. */
int64_t seg_attn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SEG_ATTN_H_ */

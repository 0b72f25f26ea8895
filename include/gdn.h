/*
 * libgdn_b200 -- chunkwise-parallel training backward of the gated delta rule (GDN) linear recurrence
 * for NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes, no framework types.
 *
 * The operation (paper Eq. 1 with one scalar gate triple per (token, head); Table 2 lists the family
 * members as gate settings).  Per (sequence n, head h) chain with state h_t of shape d_k x d_v:
 *
 *     h_t = e^{g_t} h_{t-1} + k_t (w_t v_t - b_t (e^{g_t} h_{t-1})^T k_t)^T ,     o_t = scale * h_t^T q_t
 *
 * delta_rule = 1 is GDN (erase gate b_t = write gate w_t = beta_t); delta_rule = 0 is the scalar-gate
 * linear recurrence h_t = e^{g_t} h_{t-1} + k_t v_t^T (b = 0, w = 1; beta is not read).
 * The backward differentiates  L = sum_t <dO_t, o_t> + <dhT, h_T>  and follows Section 4.2: sequences
 * are cut into chunks of 64 tokens; chunk-local WY/UT-transform factors T = (I + M)^-1 are rebuilt,
 * per-chunk states are recomputed by a forward carry, dS is propagated by a reverse carry across
 * chunks (the paper's K#1), and the intra-chunk gradients including the vector-Jacobian product of
 * the triangular solve (the paper's K#2) are formed from T without re-inverting.
 *
 * Layout (row-major, innermost last).  "dev" = device pointer, "host" = host pointer.
 *     q, k, dq, dk      dev [B, T, H, d_k]   element type desc->dtype
 *     v, dO, o, dv      dev [B, T, H, d_v]   element type desc->dtype
 *     g, beta, dg, dbeta dev [B, T, H]       float32
 *     h0, hT, dhT, dh0  dev [N, H, d_k, d_v] float32 (state orientation d_k x d_v as in Eq. 1)
 *     cu_seqlens        dev int32 [N + 1], cu[0] = 0, non-decreasing, cu[N] = T; requires B == 1.
 *                       NULL means B independent sequences of T tokens each (then N must equal B).
 * Every pointer must be 16-byte aligned.  States reset at sequence boundaries; a sequence whose length
 * is not a multiple of 64 ends in a short chunk; an empty sequence passes dhT through to dh0.
 *
 * Ownership and execution.  The caller owns every buffer; the library allocates no device memory and
 * frees nothing.  Inputs are never written.  Outputs are overwritten for every valid token.  All work
 * is enqueued on the caller's stream (a cudaStream_t passed as void*, NULL = default stream) and the
 * calls return without synchronising; cu_seqlens is never read on the host.  The workspace is scratch
 * owned by the caller; two calls may not share one workspace concurrently.  The entry points may be called
 * from several host threads at once (each call with its own workspace, on any stream): the library keeps
 * no per-call state outside the workspace, and results do not depend on what else runs on the device.
 *
 * Errors.  Argument errors are detected on the host before anything is launched and returned as a
 * status; nothing is thrown, aborted or trapped.  Conditions only visible on the device (malformed
 * cu_seqlens contents, a bounded device-side wait that ran out) are recorded in the workspace header
 * and read back by gdn_last_device_status().  Non-finite inputs propagate into the outputs.
 */
#ifndef GDN_B200_H_
#define GDN_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gdn_status {
    GDN_OK = 0,
    GDN_ERR_NULL_ARG = 1,
    GDN_ERR_BAD_SHAPE = 2,          /* non-positive dims, N inconsistent with B / cu_seqlens           */
    GDN_ERR_UNSUPPORTED_SHAPE = 3,  /* outside the envelope: chunk == 64, d_k, d_v in {64, 128}        */
    GDN_ERR_MISALIGNED = 4,         /* a pointer is not 16-byte aligned                                */
    GDN_ERR_BAD_SEQLENS = 5,        /* device-side: cu_seqlens not starting at 0 / decreasing / != T   */
    GDN_ERR_WORKSPACE_TOO_SMALL = 6,
    GDN_ERR_CUDA = 7,               /* a CUDA runtime call or launch failed                            */
    GDN_ERR_DEVICE_TIMEOUT = 8,     /* device-side: a bounded wait gave up                             */
    GDN_ERR_DECAY_RANGE = 9         /* device-side and transient: the tensor-core kernels of a channel-wise call  */
                                    /* stood down (cumulative log decay of a chunk outside [-80, 80]); the same   */
                                    /* call then runs on the FFMA kernels and clears it.  Never left behind.      */
} gdn_status;

typedef enum gdn_dtype { GDN_F32 = 0, GDN_BF16 = 1 } gdn_dtype;

typedef struct gdn_desc {
    int32_t B, T, H;      /* batch rows, tokens per row, heads                                          */
    int32_t d_k, d_v;     /* head dims, each 64 or 128                                                  */
    int32_t chunk;        /* must be 64 (Section 4.2)                                                   */
    int32_t N;            /* number of sequences: B without cu_seqlens; with cu_seqlens B must be 1     */
    int32_t dtype;        /* gdn_dtype of q, k, v, dO, o, dq, dk, dv. F32: fp32 FFMA arithmetic;        */
                          /* BF16: bf16 operands with fp32 accumulation and fp32 carried states         */
    float   scale;        /* o_t = scale * h_t^T q_t                                                    */
    int32_t delta_rule;   /* 1: b = w = beta (GDN).  0: b = 0, w = 1, beta / dbeta ignored              */
} gdn_desc;

/* Bytes of workspace needed by gdn_fwd_recompute (*fwd_bytes) and by gdn_bwd (*bwd_bytes >= *fwd_bytes;
 * the forward's workspace is a prefix of the backward's).  Either output pointer may be NULL.  Host-only
 * bookkeeping of this library (the paper has no counterpart): the workspace holds the chunk table, the
 * chunk-local factors of Section 4.2 and the per-chunk states between the stages. */
gdn_status gdn_workspace_bytes(const gdn_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes);

/* Recompute stage of the backward (Section 4.2, "chunking"): chunk table, chunk-local cumulative decay,
 * UT-transform factors T, W, U~ and the forward inter-chunk carry that leaves every chunk's incoming
 * state in the workspace.  Optionally also emits the forward outputs:
 *     o  dev [B,T,H,d_v] or NULL      hT dev [N,H,d_k,d_v] or NULL
 * beta may be NULL iff delta_rule == 0; h0 NULL means zero. */
gdn_status gdn_fwd_recompute(const gdn_desc* desc,
                             const void* q, const void* k, const void* v,
                             const float* g, const float* beta, const float* h0,
                             const int32_t* cu_seqlens_dev,
                             void* o, float* hT,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Full backward (Sections 4.1-4.2, Appendix A "the GDN backward's two hard stages").
 *     dq, dk, dv   required outputs        dg      required, gradient w.r.t. the log-decay g
 *     dbeta        required iff delta_rule dh0     optional (NULL: not written)
 *     dhT          optional (NULL = zero)  h0      optional (NULL = zero)
 * workspace_is_fresh_from_fwd != 0 asserts that `workspace` was filled by gdn_fwd_recompute with the same
 * desc, q, k, v, g, beta, h0 and cu_seqlens and not touched since; the recompute stage is then skipped. */
gdn_status gdn_bwd(const gdn_desc* desc,
                   const void* q, const void* k, const void* v,
                   const float* g, const float* beta, const float* h0,
                   const void* dO, const float* dhT,
                   const int32_t* cu_seqlens_dev,
                   void* dq, void* dk, void* dv, float* dg, float* dbeta, float* dh0,
                   void* workspace, size_t workspace_bytes, int32_t workspace_is_fresh_from_fwd,
                   void* cuda_stream);

/* ---- channel-wise gates: the general recurrence of Eq. 1 as printed ---------------------------------
 * Section 4.1, Eq. 1 and Table 2; Appendix A, "The GDN backward's two hard stages" ("the channel-wise path
 * folds the per-channel decay Diag(e^{g_t}) inside those contractions").  Three gate VECTORS per (token, head):
 *
 *     h_t = (I - k_t (b_t . k_t)^T) Diag(e^{g_t}) h_{t-1} + k_t (w_t . v_t)^T ,     o_t = scale * h_t^T q_t
 *
 *     g, b, dg, db   dev [B, T, H, d_k] float32  (log-decay and erase gate per key channel)
 *     w, dw          dev [B, T, H, d_v] float32  (write gate per value channel)
 * Every other argument, the sequence description, ownership, execution and error behaviour are those of
 * gdn_fwd_recompute / gdn_bwd; desc->delta_rule is not read (the gates say which family member runs: KDA is
 * b = w = beta broadcast over the channels, GLA is b = 0, w = 1, the full GDN has independent vectors).  All three
 * gate gradients are required outputs.  The workspace has its own size (gdn_workspace_bytes_channelwise) and
 * layout; its status word is read with gdn_last_device_status.  With bf16 I/O these calls run on the tensor cores
 * (tcgen05; kernels for d_k = d_v = 128, a head dimension of 64 is zero-padded to 128 inside the workspace, gate
 * vectors included, which is exact): keys and queries are scaled by the chunk-local cumulative decay element by element, which
 * requires |sum of g over any prefix of a 64-token chunk| <= 80 per channel; a call whose gates leave that range is
 * computed by the FFMA kernels instead (which evaluate the decay inside the contractions and have no such limit): the
 * decision is taken on the device, the call enqueues the same launches either way and needs no host round trip.  fp32
 * I/O runs on fp32 FFMA kernels throughout (with bf16 I/O they take bf16 inputs and give bf16 dq, dk, dv; all their
 * arithmetic and the gate tensors are fp32). */
gdn_status gdn_workspace_bytes_channelwise(const gdn_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes);
gdn_status gdn_fwd_recompute_channelwise(const gdn_desc* desc,
                                         const void* q, const void* k, const void* v,
                                         const float* g, const float* b, const float* w, const float* h0,
                                         const int32_t* cu_seqlens_dev,
                                         void* o, float* hT,
                                         void* workspace, size_t workspace_bytes, void* cuda_stream);
gdn_status gdn_bwd_channelwise(const gdn_desc* desc,
                               const void* q, const void* k, const void* v,
                               const float* g, const float* b, const float* w, const float* h0,
                               const void* dO, const float* dhT,
                               const int32_t* cu_seqlens_dev,
                               void* dq, void* dk, void* dv, float* dg, float* db, float* dw, float* dh0,
                               void* workspace, size_t workspace_bytes, int32_t workspace_is_fresh_from_fwd,
                               void* cuda_stream);

/* Synchronises the stream, reads the device-side status word of the last call that used `workspace`
 * and returns it (GDN_OK, GDN_ERR_BAD_SEQLENS or GDN_ERR_DEVICE_TIMEOUT; GDN_ERR_CUDA if the stream
 * itself reports an error).  Error reporting of this library (the paper has no counterpart).  After
 * a device-side error the kernels of that call stop early and leave the outputs unwritten. */
gdn_status gdn_last_device_status(const void* workspace, void* cuda_stream);

/* Static, NUL-terminated description of a status code (the paper has no counterpart). */
const char* gdn_status_string(gdn_status s);

/* Name of the kernel family a descriptor dispatches to ("simt_f32", "simt_bf16", "tcgen05_bf16",
 * "tcgen05_bf16_scalar_gate", "tcgen05_bf16_padded": bf16 shapes with one or both head dimensions at 64 that have no
 * kernels of their own, zero-padded onto the d = 128 tensor-core kernels inside the workspace),
 * or NULL for an unsupported descriptor.  Diagnostic only (the paper has no counterpart). */
const char* gdn_kernel_path(const gdn_desc* desc);
/* The same for the channel-wise calls: "tcgen05_bf16_channelwise" (bf16, d_k = d_v = 128),
 * "tcgen05_bf16_channelwise_padded" (bf16, a head dimension of 64: zero-padded onto the former inside the workspace),
 * "simt_f32_channelwise", "simt_bf16_channelwise" (the latter only under gdn_debug_force_family(1)).  Diagnostic only
 * (the paper has no counterpart); gdn_debug_force_family(1) also pins the channel-wise calls to their FFMA kernels. */
const char* gdn_kernel_path_channelwise(const gdn_desc* desc);

/* ---- backward without a caller-provided workspace (the paper has no counterpart) ----------------
 * Some callers may not allocate device memory at the point where they need the gradients: code running
 * under a memory pool that is frozen for the duration of a training step, plug-ins that are handed
 * input and output buffers by a host framework and nothing else, or processes whose memory budget was
 * fixed at start-up.  gdn_bwd_noalloc is gdn_bwd for them: same arguments without the workspace, same
 * results.  Its scratch is an array of GDN_NOALLOC_WORKSPACE_BYTES that lives inside the library on every
 * GPU that loads it, for the life of the process.  The call allocates and frees nothing.
 *   - Problems whose gdn_workspace_bytes() backward size exceeds GDN_NOALLOC_WORKSPACE_BYTES are refused
 *     with GDN_ERR_WORKSPACE_TOO_SMALL before anything is launched (at bf16, d_k = d_v = 128 the limit is
 *     about 225 chunk-heads, e.g. H = 4 and 3456 tokens).
 *   - The first call on a device looks up the array's device address (one-time set-up on the host); make
 *     that first call outside of any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents.  The call
 *     clears the part that must start from zero itself.  Two calls that overlap on the GPU (different
 *     streams, or a second call enqueued before the first has finished on another stream) race on it:
 *     keep such calls on one stream or synchronise between them.
 *   - Conditions that only the device can see (malformed cu_seqlens contents, a bounded device-side wait
 *     that ran out) make the kernels stop early: the call has returned GDN_OK by then and the outputs
 *     stay unwritten.  gdn_noalloc_last_device_status(stream) synchronises the stream and returns the
 *     status word the last gdn_bwd_noalloc on the current device left in the built-in scratch (GDN_OK,
 *     GDN_ERR_BAD_SEQLENS or GDN_ERR_DEVICE_TIMEOUT); it allocates nothing either. */
#define GDN_NOALLOC_WORKSPACE_BYTES (32u * 1024u * 1024u)
gdn_status gdn_bwd_noalloc(const gdn_desc* desc,
                           const void* q, const void* k, const void* v,
                           const float* g, const float* beta, const float* h0,
                           const void* dO, const float* dhT,
                           const int32_t* cu_seqlens_dev,
                           void* dq, void* dk, void* dv, float* dg, float* dbeta, float* dh0,
                           void* cuda_stream);
gdn_status gdn_noalloc_last_device_status(void* cuda_stream);

/* ---- measurement hooks (not part of the method; the paper has no counterpart) -------------------
 * gdn_launch_count: number of kernels this library has launched in this process.
 * gdn_stage_timing_enable(n), n >= 1: from now on every kernel launch of every n-th call of gdn_fwd_recompute /
 * gdn_bwd (the first one included) is bracketed by a pair of CUDA events recorded on the launching stream (events
 * are created lazily and reused; no device memory).  An event between two kernels costs the stream a few
 * microseconds, which is why a timed loop samples (n > 1) instead of bracketing every launch.  0 switches it off.
 * gdn_stage_timing_read: synchronises the recorded events, adds up per-stage durations since the last
 * read, writes up to max_stages entries (total_ms, launches, names: static strings) and resets the
 * record.  Returns the number of stages through *n_stages.  Not thread-safe; diagnostic use only. */
uint64_t gdn_launch_count(void);
gdn_status gdn_stage_timing_enable(int32_t on);
gdn_status gdn_stage_timing_read(int32_t max_stages, float* total_ms, int32_t* launches, const char** names,
                                 int32_t* n_stages);

/* ---- debugging hooks (the paper has no counterpart) ---------------------------------------------
 * gdn_debug_read: synchronises the device and copies one workspace quantity of one (chunk, head) to
 * host memory as row-major float32, whatever the internal storage format:
 *   "gamma" [64]   "T" [64,64]   "W" [64,d_k]   "Ut" [64,d_v]   "Nm" [d_k,d_k]
 *   "Bf", "E", "hc", "dhn" [d_k,d_v]
 * "Nm" and "Bf" are written only when the carries run in operator form (see below).
 * gdn_debug_force_family: 0 = automatic dispatch, 1 = always use the FFMA kernels (tests use this to
 * exercise both families on the same inputs); 2 / 3 = automatic family, but the tcgen05 d = 128 kernels carry the
 * state across chunks in operator form (one d x d matrix per chunk) / in low-rank form (two dependent products
 * per chunk, no such matrix), whatever the shape; by default the shape decides.  The setting belongs to the
 * calling thread (other threads keep automatic dispatch) and changes what gdn_workspace_bytes returns to that thread,
 * so size the workspace after setting it. */
gdn_status gdn_debug_read(const gdn_desc* desc, const void* workspace, const char* what, int32_t chunk, int32_t head,
                          float* host_out);
gdn_status gdn_debug_force_family(int32_t family);
/* gdn_debug_inject_timeout(1): the next gdn_bwd of the calling thread that runs on the tcgen05 d = 128 family (and
 * recomputes the forward) exercises the library's failure path without faulting anything: for that one call the
 * bounded device-side waits give up after a millisecond instead of two seconds, and the first chunk-level kernel
 * leaves out one of its input loads, so the wait for it runs out.  The CTAs leave through their normal teardown
 * (tensor memory released, no copy in flight), the remaining kernels of the call see the status word and write
 * nothing, gdn_bwd itself returns GDN_OK and gdn_last_device_status reports GDN_ERR_DEVICE_TIMEOUT.  The next call
 * is a normal one.  0 cancels a pending request. */
gdn_status gdn_debug_inject_timeout(int32_t on);

#ifdef __cplusplus
}
#endif
#endif /* GDN_B200_H_ */

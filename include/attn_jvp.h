/*
 * attn_jvp.h -- C ABI of the B200 (sm_100a) attention-JVP library.
 *
 * One operation: the forward-mode Jacobian-vector product of non-causal
 * softmax attention, fused into a single streaming pass over the keys
 * (Appendix C.1 "FlashAttention-2 JVP", Algorithm 2).  For every batch b and
 * head h independently, with s = `scale`:
 *
 *     S  = s Q K^T                P  = softmax_rows(S)          O = P V
 *     tS = s (tQ K^T + Q tK^T)    mu = rowsum(P . tS)
 *     tO = (P . tS) V + P tV - diag(mu) O                       (aggregated form, Appendix C.1)
 *     LSE_i = log sum_j exp(S_ij)                               (Algorithm 2, L = m + log l)
 *
 * The paper writes S = Q K^T without a softmax scale; here the constant
 * `scale` multiplies both S and tS and is not differentiated.
 *
 * Conventions common to every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller.  The
 *     library neither frees nor retains them and allocates no device memory;
 *     the split-KV and the host-buffer entry points need a (caller-provided)
 *     device workspace, all others need none.
 *   - q, tq, o, to : bf16, layout [B][Lq][H][D] contiguous ("BLHD").
 *     k, v, tk, tv : bf16, layout [B][Lk][H][D] contiguous.
 *     lse          : fp32, layout [B][H][Lq], natural log of the scaled scores.
 *   - D is 64 or 128.  Lq and Lk are arbitrary positive lengths (no multiple
 *     of the tile size is required).  Same H for queries and keys.
 *   - Arithmetic: bf16 operands, fp32 accumulation, outputs rounded to bf16
 *     (round to nearest even).  Inputs are assumed finite.
 *   - Calls are asynchronous: work is enqueued on a CUDA stream and the
 *     function returns.  Rows i >= Lq are never written.
 *   - Return value: 0 on success, otherwise one of the ATTN_JVP_ERR_* codes
 *     below, in which case NOTHING has been enqueued.  No exceptions, no
 *     exit(), no CPU fallback.
 *   - Every device-side wait is bounded.  If one expires (a bug, never expected)
 *     the kernel stops early and records ATTN_JVP_ERR_DEVICE_TIMEOUT, which
 *     attn_jvp_device_status() reports after the caller has synchronised.
 */
#ifndef ATTN_JVP_H_
#define ATTN_JVP_H_

#ifdef __cplusplus
extern "C" {
#endif

/* flags */
#define ATTN_JVP_KV_TANGENT_FREE 0x1u /* tK = tV = 0 (cross-attention on a constant context,  */
                                      /* Sec. 3.2 / Appendix C.2); tk, tv ignored, may be NULL */
#define ATTN_JVP_FWD_ONLY        0x2u /* plain forward of the same kernel: only O and LSE are  */
                                      /* produced; tq, tk, tv, to ignored, may be NULL         */

/* error codes */
#define ATTN_JVP_OK                  0
#define ATTN_JVP_ERR_NULL            1  /* a required pointer is NULL */
#define ATTN_JVP_ERR_SHAPE           2  /* B, H, Lq or Lk < 1; sizes or the work-item count overflow; bad splits / heads_per_stage */
#define ATTN_JVP_ERR_UNSUPPORTED_D   3  /* D is not 64 or 128 */
#define ATTN_JVP_ERR_ALIGN           4  /* a tensor pointer is not 16-byte aligned */
#define ATTN_JVP_ERR_FLAGS           5  /* unknown flag bits */
#define ATTN_JVP_ERR_SCALE           6  /* scale is NaN or infinite */
#define ATTN_JVP_ERR_ALIAS           7  /* an output buffer overlaps an input or another output */
#define ATTN_JVP_ERR_ARCH            8  /* current device is not compute capability 10.x */
#define ATTN_JVP_ERR_CUDA            9  /* a CUDA runtime / driver call failed (see strerror) */
#define ATTN_JVP_ERR_DEVICE_TIMEOUT 10  /* a bounded device-side wait expired */
#define ATTN_JVP_ERR_DEVICE_LAYOUT  11  /* the kernel's shared-memory layout did not fit (reported like a timeout) */
#define ATTN_JVP_ERR_WORKSPACE      12  /* the caller's workspace is too small */
#define ATTN_JVP_ERR_STATIC_SCRATCH 13  /* the call needs more scratch than ATTN_JVP_STATIC_SCRATCH_BYTES */

/* Size of the scratch buffer built into the library for attn_jvp_fwd_splitkv_static (32 MiB). */
#define ATTN_JVP_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)

/*
 * attn_jvp_fwd -- O, tO and LSE of Algorithm 2 in one pass, on the stream set
 * by attn_jvp_set_stream (default: the legacy default stream).
 *
 *   q,k,v,tq,tk,tv  inputs (device, bf16 BLHD).  With ATTN_JVP_KV_TANGENT_FREE
 *                   tk and tv are not read.  With ATTN_JVP_FWD_ONLY tq, tk, tv
 *                   are not read and `to` is not written.
 *   o, to           outputs (device, bf16 BLHD, [B][Lq][H][D]).
 *   lse             output (device, fp32 [B][H][Lq]).
 *   B,H,Lq,Lk,D     sizes; scale: softmax scale s; flags: ATTN_JVP_* bits.
 */
int attn_jvp_fwd(const void* q, const void* k, const void* v,
                 const void* tq, const void* tk, const void* tv,
                 void* o, void* to, float* lse,
                 int B, int H, int Lq, int Lk, int D,
                 float scale, unsigned flags);

/* Same operation (Algorithm 2) on an explicit CUDA stream (a cudaStream_t passed as void*). */
int attn_jvp_fwd_stream(const void* q, const void* k, const void* v,
                        const void* tq, const void* tk, const void* tv,
                        void* o, void* to, float* lse,
                        int B, int H, int Lq, int Lk, int D,
                        float scale, unsigned flags, void* cuda_stream);

/*
 * attn_jvp_fwd_mu -- Algorithm 2 plus one more per-row side output, mu = rowsum(P . tS) (the r / l of
 * Algorithm 2 lines 16 and 21, i.e. the tangent of L = LSE).  mu: device, fp32 [B][H][Lq], required.
 * Everything else as attn_jvp_fwd_stream.  With ATTN_JVP_FWD_ONLY mu is written as 0.
 */
int attn_jvp_fwd_mu(const void* q, const void* k, const void* v,
                    const void* tq, const void* tk, const void* tv,
                    void* o, void* to, float* lse, float* mu,
                    int B, int H, int Lq, int Lk, int D,
                    float scale, unsigned flags, void* cuda_stream);

/*
 * Split-KV variant for few queries and many keys: the keys are cut into chunks of whole 64-key tiles,
 * each (query tile, head, chunk) runs Algorithm 2 on its chunk, and a second kernel merges the chunks.
 * With per-chunk results (O_c, tO_c, LSE_c, mu_c) and w_c = exp(LSE_c - LSE), LSE = log sum_c exp(LSE_c):
 *     O = sum_c w_c O_c,  mu = sum_c w_c mu_c,  tO = sum_c w_c (tO_c + mu_c O_c) - mu O,
 * which is the aggregated form of Appendix C.1 regrouped by chunk (exact in real arithmetic).
 *
 *   splits           requested number of chunks (>= 1); the library uses ceil(tiles / ceil(tiles / splits))
 *                    chunks so that none is empty; 1 chunk = the plain kernel, no workspace needed.
 *   workspace        device scratch owned by the caller, 16-byte aligned, at least
 *                    attn_jvp_splitkv_workspace_bytes(...) bytes; contents undefined afterwards.  Calls
 *                    that share a workspace must not overlap on the GPU.
 *   mu               optional (may be NULL).  Other arguments as attn_jvp_fwd_stream.
 * Returns ATTN_JVP_ERR_WORKSPACE if workspace_bytes is too small.
 */
size_t attn_jvp_splitkv_workspace_bytes(int B, int H, int Lq, int Lk, int D, int splits);
/* A number of chunks for attn_jvp_fwd_splitkv that fills the current device: 1 when the query tiles alone keep
 * at least ~60 % of the SMs busy, else the largest count for which (query tiles x heads x batch x chunks) still
 * fits one wave of CTAs, with at least four 64-key tiles per chunk.  (A heuristic of this library, measured on
 * B200; the paper has no counterpart.)  Returns 1 for invalid shapes or when no CUDA device is current. */
int attn_jvp_suggest_splits(int B, int H, int Lq, int Lk, int D);
int attn_jvp_fwd_splitkv(const void* q, const void* k, const void* v,
                         const void* tq, const void* tk, const void* tv,
                         void* o, void* to, float* lse, float* mu,
                         int B, int H, int Lq, int Lk, int D,
                         float scale, unsigned flags, int splits,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * attn_jvp_fwd_host -- the operation of attn_jvp_fwd_stream (Appendix C.1 / Algorithm 2) on HOST tensors.
 *
 * q, k, v, tq, tk, tv, o, to, lse are HOST pointers with the layouts of attn_jvp_fwd (bf16 [B][L][H][D], LSE fp32
 * [B][H][Lq]); page-locked (pinned) memory is needed for the copies to overlap with the kernel, pageable memory
 * works but is copied synchronously.  The heads are processed in groups of `heads_per_stage`: the group's heads
 * are gathered out of the interleaved host rows into a dense device copy ([B][L][heads][D]), the kernel runs on
 * that copy, and its O, tO, LSE are scattered back to the host tensors, while the copy engines already move the
 * next group in and the previous group out.  Every (b, h) is computed exactly as by attn_jvp_fwd on a device
 * tensor (the result of a head does not depend on the other heads), so the outputs are bit-identical.
 *
 *   heads_per_stage  heads per pipeline stage; 0 = library default (about ten stages where the kernel takes as
 *                    long as the copies, about five where the copies set the pace; copy rows >= 512 bytes).
 *   workspace        DEVICE scratch owned by the caller, 256-byte aligned, at least
 *                    attn_jvp_host_workspace_bytes(...) bytes (three buffer sets of one head group: eight bf16
 *                    tensors and the LSE block); contents undefined afterwards.  Two calls that share a
 *                    workspace must be ordered on the GPU (same stream, or an event between their streams).
 *   cuda_stream      the work is ordered after what is already on this stream, and the stream continues only
 *                    after the last output byte has reached the host; the copies and the kernel themselves run
 *                    on three streams the library creates once per device.  The call returns when everything is
 *                    enqueued: host inputs must stay unchanged, and host outputs unread, until the stream has
 *                    been synchronised.  Calls on one device are serialised on the host by a lock.
 * Flags, scale and error codes as attn_jvp_fwd; ATTN_JVP_ERR_WORKSPACE if workspace_bytes is too small,
 * ATTN_JVP_ERR_ALIGN if the workspace is not 256-byte aligned.  Nothing is enqueued unless the arguments check
 * out; if a CUDA call fails part-way, what was enqueued still completes before the stream continues.
 */
size_t attn_jvp_host_workspace_bytes(int B, int H, int Lq, int Lk, int D, int heads_per_stage);
int attn_jvp_fwd_host(const void* q, const void* k, const void* v,
                      const void* tq, const void* tk, const void* tv,
                      void* o, void* to, float* lse,
                      int B, int H, int Lq, int Lk, int D,
                      float scale, unsigned flags, int heads_per_stage,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * attn_jvp_fwd_splitkv_static -- the split-KV computation of attn_jvp_fwd_splitkv for callers that are not
 * allowed to allocate GPU memory.  (No counterpart in the paper: this is a packaging variant, the arithmetic
 * is that of attn_jvp_fwd_splitkv.)
 *
 * Who needs it: code that runs where a cudaMalloc is off limits -- a real-time or serving loop whose memory was
 * fixed at start-up and which cannot afford the device-wide synchronisation an allocation implies, a framework
 * whose allocator must own every byte, or a process whose memory budget is already spent.  Such
 * a caller cannot provide the workspace that attn_jvp_fwd_splitkv asks for, so this entry point brings its own:
 * a fixed array of ATTN_JVP_STATIC_SCRATCH_BYTES (32 MiB) that is part of the library's device image.  Every GPU
 * on which the library is loaded gives up that much memory until the process exits, whether or not this
 * function is ever called.
 *
 * Behaviour
 *   - Arguments as attn_jvp_fwd_splitkv, without workspace / workspace_bytes.  Inputs and outputs are still the
 *     caller's device buffers.
 *   - The function itself calls no cudaMalloc / cudaFree / cudaHostAlloc and no allocating library routine.
 *     (It also skips the pinned status word the other entry points create on first use; a device-side timeout in
 *     a call made before any other entry point ran on this device is then only visible as later launches
 *     returning at once.)
 *   - A call whose chunks need more than ATTN_JVP_STATIC_SCRATCH_BYTES (see attn_jvp_splitkv_workspace_bytes)
 *     is refused with ATTN_JVP_ERR_STATIC_SCRATCH and nothing is enqueued; attn_jvp_strerror gives both sizes.
 *   - The first call on each device looks up the array's device address (with that device current), and the
 *     first call per (D, flags) combination sets a launch attribute of the kernel it selects.  Make these first
 *     calls before any stream capture begins.
 *   - All calls on a device share the one array and it keeps whatever the previous call left in it.  Nothing in
 *     it has to start at zero: every value that the merge step reads is written by the same call first.  Two calls
 *     that overlap on the GPU (different streams, no dependency between them) race on the array and produce
 *     garbage; calls on one stream, or otherwise ordered, are fine.
 */
int attn_jvp_fwd_splitkv_static(const void* q, const void* k, const void* v,
                                const void* tq, const void* tk, const void* tv,
                                void* o, void* to, float* lse, float* mu,
                                int B, int H, int Lq, int Lk, int D,
                                float scale, unsigned flags, int splits, void* cuda_stream);

/*
 * Tuning knobs for benchmarking and A/B comparisons (process-wide; the paper has no counterpart).  Every setting
 * computes the same function within the library's tolerance; only the kernel variant changes.
 *   ATTN_JVP_TUNE_SOFTMAX_GROUPS  0 = the library chooses per (mode, D, keys) (default), 1 = one softmax warpgroup
 *                                 per CTA plus a warpgroup that runs the work items' epilogues, 2 = two softmax
 *                                 warpgroups taking alternate key tiles (384 threads either way).
 *   ATTN_JVP_TUNE_CTA_PAIR        0 = the library chooses (default), 1 = never, 2 = whenever it exists (D = 128, no
 *                                 key chunks): the kernel variant in which two CTAs on neighbouring SMs share a
 *                                 256-row query block, the K/V operand tiles and one MMA instruction stream.
 * Returns 0, or ATTN_JVP_ERR_FLAGS for an unknown knob or value.
 */
#define ATTN_JVP_TUNE_SOFTMAX_GROUPS 1
#define ATTN_JVP_TUNE_CTA_PAIR 2
int attn_jvp_set_tuning(int knob, int value);

/*
 * Diagnostics after ATTN_JVP_ERR_DEVICE_TIMEOUT (a bug report aid; the paper has no counterpart): which bounded
 * wait gave up first on the current device since the last call.  out[0..3] (host memory) receive the
 * shared-memory address of the barrier, the phase parity waited for, threadIdx.x and blockIdx.x of the waiting
 * thread.  Returns 1 if there was a record (it is cleared), 0 if none, -1 on a CUDA error or NULL.  Blocking.
 */
int attn_jvp_debug_timeout_info(unsigned* out);

/* Sets the stream attn_jvp_fwd launches on for the calling host thread
 * (thread-local; NULL = legacy default stream).  Always returns 0. */
int attn_jvp_set_stream(void* cuda_stream);

/*
 * Device-side status of the current device since the last call of this
 * function: 0, or ATTN_JVP_ERR_DEVICE_TIMEOUT if a bounded wait inside a
 * kernel expired (ATTN_JVP_ERR_DEVICE_LAYOUT if its shared-memory layout did
 * not fit).  Meaningful once the caller has synchronised the stream(s) the
 * kernels ran on; reading it clears it (and lets later launches run again).
 * Normally this only reads a pinned host word.  It copies a word from the
 * device (and so orders itself after work on the legacy default stream) only
 * after a reported timeout, or while attn_jvp_fwd_splitkv_static is the only
 * entry point that has run on the device; it never waits for other streams.
 */
int attn_jvp_device_status(void);

/*
 * attn_jvp_qknorm_fwd -- RMS normalisation over the head dimension together with its forward-mode tangent,
 * the step that produces q, k, tq, tk for the attention kernel in a DiT block with QK normalisation (Sec. 3.1;
 * Appendix C.2 restructures an RMSNorm layer for JVP mode).  Per row x in R^D, with frozen weight w:
 *     n = sqrt(mean(x^2) + eps),   y = w . x / n,   ty = w . (tx / n - x (x . tx) / (D n^3)).
 *
 *   x, tx   device, bf16, `rows` rows of D contiguous elements (any [..][D] layout, e.g. [B][L][H][D]);
 *           tx may be NULL together with ty (primal only).
 *   w       device, fp32 [D].      y, ty   device, bf16, same shape as x.
 *   rows >= 1; D is 64 or 128; eps >= 0; all pointers 16-byte aligned; outputs must not overlap inputs.
 * Asynchronous on `cuda_stream`; returns 0 or an ATTN_JVP_ERR_* code (nothing enqueued on error).
 */
int attn_jvp_qknorm_fwd(const void* x, const void* tx, const float* w, void* y, void* ty,
                        long long rows, int D, float eps, void* cuda_stream);

/*
 * Self-test of the failure path (no counterpart in the paper): enqueues a one-warp kernel that waits on a
 * barrier nothing ever signals.  The wait expires after its time limit (about 2 s), the kernel ends normally,
 * and attn_jvp_device_status() then reports ATTN_JVP_ERR_DEVICE_TIMEOUT, exactly as it would for a stalled
 * attention kernel.  Nothing is trapped or faulted; the device stays usable.  Returns 0 when enqueued.
 */
int attn_jvp_selftest_bounded_wait(void* cuda_stream);

/* Human-readable text for a return code; for ATTN_JVP_ERR_CUDA the text of the
 * last failing CUDA call on this thread is appended.  Never NULL. */
const char* attn_jvp_strerror(int code);

/* Library version: major*10000 + minor*100 + patch. */
int attn_jvp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ATTN_JVP_H_ */

/*
 * laga.h -- C ABI of the B200 (sm_100a) LAGA per-rank attention hot path.
 *
 * What the library computes.  One sequence-parallel rank's work after the latent all-gather of
 * LAGA (paper Algorithm 1, steps 4 and 5) and its backward (paper Section 5.2):
 *
 *   step 4   KV = c_kv . W_kv_b[H_r]                (head-shard up-projection of the gathered latent)
 *            K_nope[t,i,:] = KV[t, i*(d_nope+d_v) + 0 .. d_nope)
 *            V[t,i,:]      = KV[t, i*(d_nope+d_v) + d_nope .. d_nope+d_v)
 *   step 5   K[t,i,:] = K_nope[t,i,:] || k_pe[t,:]   (the rope key band is shared by all heads, Sec. 2.1)
 *            scores = softmax_scale * q K^T, masked to t <= s when causal
 *            O = softmax(scores) V,   LSE = natural-log-sum-exp of the masked scaled scores
 *   backward dQ, dc_kv (partial sum over this head shard), dk_pe (sum over this head shard) and
 *            dW_kv_b[H_r] (complete for these heads: the "(full_seq, H_r)" gradient shard of Sec. 5.2)
 *
 * Conventions common to every call
 *   - Every data pointer is a DEVICE pointer owned by the caller; the library allocates nothing,
 *     frees nothing and keeps no pointer after the call returns.  Buffers must stay valid until the
 *     work enqueued on `stream` has finished.  All base pointers must be 16-byte aligned.
 *   - All tensors are dense row-major ("C order") with the shapes given below; bf16 tensors are
 *     passed as `const void*` / `void*` pointing at 16-bit brain-float elements.
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*; NULL is the default
 *     stream) and return without synchronising, except laga_query_status.
 *   - Return value: LAGA_OK (0) or a negative LAGA_ERR_* code.  Argument errors are detected before
 *     anything is enqueued.  Nothing throws, aborts or traps.
 *   - Work runs on the CURRENT device (cudaSetDevice): every data pointer must be device memory of that
 *     device (or managed memory); a pointer that belongs to another device, or to the host, returns
 *     LAGA_ERR_INVALID_ARG before anything is enqueued.
 *   - The entry points may be called from several host threads at once (the library's per-device and
 *     tensor-map caches are locked); what the callers must keep apart is the memory: two calls that may
 *     overlap on the GPU must not share a workspace or an output.
 *   - This build is written for the DeepSeek-V3 head geometry: d_nope = 128, d_rope = 64, d_v = 128 (the
 *     attention kernels' tiles and TMEM maps); other head dimensions return LAGA_ERR_UNSUPPORTED.  The latent
 *     width d_c is free: any multiple of 8 from 8 to 8192 (it only enters the three token-wise GEMMs); 512 is
 *     the tuned and benchmarked value.  The absorbed comparison form and LAGA_FLAG_FUSED_KV_REBUILD need
 *     d_c = 512.  S >= 1 and h >= 1 are arbitrary (S need not be a multiple of any tile).  Batches: the
 *     _varlen entry points.
 *   - `workspace` is caller-provided scratch of at least laga_*_workspace_bytes(...) bytes, 1024-byte
 *     aligned.  Its first 1024 bytes are the launch status slot (the status word laga_query_status reads,
 *     the work counters of the persistent kernels, their clock probes); every call clears what it needs.
 */
#ifndef LAGA_H_
#define LAGA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LAGA_OK 0
#define LAGA_ERR_INVALID_ARG (-1)         /* NULL or misaligned pointer, S < 1, h < 1, bad flag     */
#define LAGA_ERR_UNSUPPORTED (-2)         /* head geometry other than 128/64/128 (see above), or not sm_100 */
#define LAGA_ERR_WORKSPACE_TOO_SMALL (-3)
#define LAGA_ERR_CUDA (-4)                /* a CUDA runtime/driver call or a launch failed          */
#define LAGA_ERR_DEVICE_TIMEOUT (-5)      /* only from laga_query_status: a bounded device wait ran out */
#define LAGA_ERR_DEVICE_CHECK (-6)        /* only from laga_query_status: a device-side self-check failed
                                             (the kernel recorded where, skipped the access and returned)   */

#define LAGA_FLAG_ACCUM_DW 1u             /* laga_bwd: add into dw_kv_b instead of overwriting it   */
#define LAGA_FLAG_DETERMINISTIC 2u        /* laga_bwd: bitwise-repeatable dk_pe and dw_kv_b (see there) */
#define LAGA_FLAG_KV_SAVED 4u             /* laga_bwd: the workspace still holds laga_fwd's K_nope/V (see there) */
#define LAGA_FLAG_FUSED_BWD 8u            /* laga_bwd: one-pass backward attention on CTA pairs (see there)       */
#define LAGA_FLAG_FUSED_KV_REBUILD 16u    /* laga_bwd: step 4 rebuilt inside the dK/dV kernel (see there)         */

/* Library version (major*10000 + minor*100 + patch). */
int laga_version(void);

/* Static, human-readable name of a status code. */
const char* laga_status_string(int status);

/* Scratch sizes in bytes for the calls below (0 if the geometry is unsupported). */
size_t laga_fwd_workspace_bytes(int S, int h, int d_c, int d_nope, int d_rope, int d_v);
size_t laga_bwd_workspace_bytes(int S, int h, int d_c, int d_nope, int d_rope, int d_v, unsigned flags);

/*
 * Forward: Algorithm 1 steps 4-5.
 *   q       bf16 [S, h, d_nope+d_rope]   queries of this head shard, nope band first, rope band last
 *                                        (already rotated)
 *   c_kv    bf16 [S, d_c]                gathered, already-normalised latent
 *   k_pe    bf16 [S, d_rope]             gathered, already-rotated shared rope key
 *   w_kv_b  bf16 [d_c, h*(d_nope+d_v)]   head shard of W_kv_b; column i*(d_nope+d_v)+j is K_nope
 *                                        channel j of head i for j < d_nope, else V channel j-d_nope
 *   out     bf16 [S, h, d_v]             written
 *   lse     fp32 [S, h]                  written
 * `causal` != 0 masks keys t > s.  The per-head K_nope/V are materialised in bf16 inside `workspace`
 * (the explicit form's own footprint); nothing else of size S x S or S x h x d_c exists.
 */
int laga_fwd(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, int S, int h, int d_c,
             int d_nope, int d_rope, int d_v, float softmax_scale, int causal, void* out, float* lse,
             void* workspace, size_t workspace_bytes, unsigned flags, void* stream);

/*
 * Backward: Section 5.2 (chain rule through step 5, then back through step 4).
 *   q, c_kv, k_pe, w_kv_b   as in laga_fwd
 *   out, lse                what laga_fwd produced for the same inputs
 *   dout    bf16 [S, h, d_v]             upstream gradient of out
 *   dq      bf16 [S, h, d_nope+d_rope]   written
 *   dc_kv   bf16 [S, d_c]                written: this head shard's contribution (ranks reduce-scatter it)
 *   dk_pe   bf16 [S, d_rope]             written: summed over this shard's heads
 *   dw_kv_b fp32 [d_c, h*(d_nope+d_v)]   overwritten, or accumulated into with LAGA_FLAG_ACCUM_DW
 * K_nope/V are recomputed from c_kv (the forward keeps only out and lse).  All accumulation is fp32.
 * dw_kv_b (over the sequence) and dk_pe (over the heads) are reduced with floating-point atomics:
 * their low-order bits may differ from run to run.  LAGA_FLAG_DETERMINISTIC removes that: dw_kv_b is
 * then computed without splitting the sequence (one addition per element; fewer CTAs, so the dW GEMM
 * is slower) and dk_pe is summed over per-head buffers in head order (S*h*d_rope*4 more workspace
 * bytes: pass the same flags to laga_bwd_workspace_bytes).  dq and dc_kv are repeatable either way.
 * LAGA_FLAG_KV_SAVED skips the recomputation of step 4: it promises that laga_fwd ran on the same
 * c_kv and w_kv_b with this very workspace pointer (sized by laga_bwd_workspace_bytes) and that nothing
 * has written to the workspace since -- the forward leaves K_nope/V where the backward looks for them.
 * This is the explicit form's way of saving K/V for the backward; the price is that the workspace cannot
 * be shared with another layer between the two calls.  The library cannot check the promise.
 * LAGA_FLAG_FUSED_BWD selects the one-pass backward attention: clusters of two CTAs compute each score
 * tile once (one CTA scores, softmax and dV; its peer dK and dQ from the dS tile it receives through
 * distributed shared memory) and dQ is summed over key tiles in an fp32 accumulator with atomic additions
 * (S * w * 192 * 4 more workspace bytes for a window of w heads, at most 64 MB: pass the flag to
 * laga_bwd_workspace_bytes), so dq is then not repeatable bit for bit.  It executes 5 instead of 7 tile
 * products but is the SLOWER path on B200 as measured (its exponentials sit on one of the two SMs); it is
 * not the default and cannot be combined with LAGA_FLAG_DETERMINISTIC (LAGA_ERR_INVALID_ARG).
 * LAGA_FLAG_FUSED_KV_REBUILD fuses the recomputation of step 4 into the dK/dV kernel (the open direction the
 * paper names in Section 4.7: a fused up-projection -> attention kernel): every (key tile, head) item builds its
 * own K_nope / V tile from c_kv and the head's block of w_kv_b with tensor-core MMAs in its prologue and stores
 * it to the workspace for the dQ kernel; the separate up-projection launch is dropped.  Same results (bit for bit
 * with LAGA_FLAG_DETERMINISTIC on both sides); same workspace; one launch less.  Not combinable with LAGA_FLAG_KV_SAVED
 * or LAGA_FLAG_FUSED_BWD (LAGA_ERR_INVALID_ARG).  Measured on B200: within 3 % of the default path from S = 512 to
 * S = 16384 (what the saved launch gains, the prologue -- serial work per item: the accumulators it builds the
 * tile in are free only between the previous item's drain and this item's first product -- gives back); opt-in.
 */
int laga_bwd(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, const void* out,
             const float* lse, const void* dout, int S, int h, int d_c, int d_nope, int d_rope, int d_v,
             float softmax_scale, int causal, void* dq, void* dc_kv, void* dk_pe, float* dw_kv_b,
             void* workspace, size_t workspace_bytes, unsigned flags, void* stream);

/*
 * Batches and variable-length sequences (Algorithm 1 steps 4-5 and Section 5.2 applied per sequence).
 *
 * n_seqs sequences are PACKED along the token axis: q [S_total, h, 192], c_kv [S_total, d_c], k_pe [S_total, d_rope]
 * and every output in the same row order, sequence k occupying rows cu_seqlens[k] .. cu_seqlens[k+1]-1.
 * cu_seqlens is a HOST array of n_seqs + 1 non-decreasing integers with cu_seqlens[0] = 0 and
 * cu_seqlens[n_seqs] = S_total (a batch of B equal sequences of length L is {0, L, 2L, ...}; empty sequences are
 * allowed).  Attention (and its causal mask) is confined to each sequence; the projections of step 4 and of
 * Section 5.2 are token-wise and run once over all the packed tokens; dw_kv_b sums over all sequences, dk_pe
 * over the shard's heads as in laga_bwd.  Everything else -- layouts, dtypes, flags, errors, ownership -- is as
 * for laga_fwd / laga_bwd, with these differences:
 *   - the workspace is sized by the _varlen_ queries below (they need n_seqs, not the lengths); LAGA_FLAG_KV_SAVED
 *     pairs laga_fwd_varlen with laga_bwd_varlen on the same workspace, cu_seqlens included;
 *   - the call copies a small table (32 bytes per 128-token tile) from host memory into the workspace, which
 *     makes it synchronise with the stream's earlier work and unsuitable for CUDA-graph capture;
 *   - LAGA_FLAG_FUSED_BWD is not available (LAGA_ERR_INVALID_ARG; its workspace query returns 0).
 * A malformed cu_seqlens (not starting at 0, decreasing, not ending at S_total, or no token at all) is
 * LAGA_ERR_INVALID_ARG before anything is enqueued.  All sequences' tiles are handed to the persistent kernels
 * in one launch each, longest first.
 */
size_t laga_fwd_varlen_workspace_bytes(int S_total, int n_seqs, int h, int d_c, int d_nope, int d_rope, int d_v);
size_t laga_bwd_varlen_workspace_bytes(int S_total, int n_seqs, int h, int d_c, int d_nope, int d_rope, int d_v,
                                       unsigned flags);
int laga_fwd_varlen(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, const int* cu_seqlens,
                    int n_seqs, int S_total, int h, int d_c, int d_nope, int d_rope, int d_v, float softmax_scale,
                    int causal, void* out, float* lse, void* workspace, size_t workspace_bytes, unsigned flags,
                    void* stream);
int laga_bwd_varlen(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, const void* out,
                    const float* lse, const void* dout, const int* cu_seqlens, int n_seqs, int S_total, int h,
                    int d_c, int d_nope, int d_rope, int d_v, float softmax_scale, int causal, void* dq, void* dc_kv,
                    void* dk_pe, float* dw_kv_b, void* workspace, size_t workspace_bytes, unsigned flags,
                    void* stream);

/*
 * The dense projections around the path (Algorithm 1 steps 1 and 7: W_q, W_kv_a, W_o), on the same CTA-pair
 * tcgen05 GEMM that runs step 4.  All bf16, row-major, device pointers; fp32 accumulation.
 *
 * laga_linear:           y bf16 [M, N] = x [M, K] . w [K, N]
 * laga_linear_backward:  dx bf16 [M, K] = dy [M, N] . w^T          written
 *                        dw fp32 [K, N] (+)= x^T . dy               overwritten, or added to with LAGA_FLAG_ACCUM_DW;
 *                        LAGA_FLAG_DETERMINISTIC as for laga_bwd (no split over M, one addition per element)
 * M >= 1 is arbitrary; K and N must be multiples of 8 (row pitches of 16 bytes), anything else is
 * LAGA_ERR_INVALID_ARG.  N and K need not be multiples of the 256-column tiles (576 works).
 * status_word: one device word (4 bytes, 4-byte aligned), cleared by the call; read it with laga_query_status.
 */
int laga_linear(const void* x, const void* w, int M, int K, int N, void* y, void* status_word, void* stream);
int laga_linear_backward(const void* dy, const void* x, const void* w, int M, int K, int N, void* dx, float* dw,
                         unsigned flags, void* status_word, void* stream);

/*
 * LayerNorm of the latent (Algorithm 1 step 1: latent <- LayerNorm(latent), between W_kv_a and the gather).
 * The paper names the operation and nothing else; this is the usual definition over the last axis with
 * biased variance, learnable scale and optional shift:
 *   y[m, :] = (x[m, :] - mean_m) * rstd_m * gamma + beta,   rstd_m = 1 / sqrt(var_m + eps)
 * x, y, dy, dx bf16 [M, D]; gamma, beta bf16 [D] (beta may be NULL: no shift); statistics and arithmetic fp32.
 * laga_layernorm optionally writes mean and rstd (fp32 [M]; either may be NULL) -- the backward needs both.
 * laga_layernorm_backward writes dx and OVERWRITES dgamma fp32 [D] and, if not NULL, dbeta fp32 [D] (sums over
 * the M rows, added with fp32 atomics: low-order bits may vary from run to run).
 * D must be a multiple of 8 and at most 1024 (the latent is 512 wide), eps >= 0; anything else is
 * LAGA_ERR_INVALID_ARG.  HBM-bound kernels without bounded waits: no status word, errors are launch errors.
 */
int laga_layernorm(const void* x, const void* gamma, const void* beta, int M, int D, float eps, void* y, float* mean,
                   float* rstd, void* stream);
int laga_layernorm_backward(const void* dy, const void* x, const void* gamma, const float* mean, const float* rstd, int M,
                            int D, void* dx, float* dgamma, float* dbeta, void* stream);

/*
 * Step entry points (the same kernels laga_fwd / laga_bwd launch, callable on their own).
 *
 * laga_up_project: Algorithm 1 step 4.   kv bf16 [S, h*(d_nope+d_v)] = c_kv . w_kv_b  (fp32 accumulate).
 * laga_kv_backward: Section 5.2, back through step 4.  Given dkv bf16 [S, h*(d_nope+d_v)] (per head:
 *   dK_nope then dV), writes dc_kv bf16 [S, d_c] = dkv . w_kv_b^T and dw_kv_b fp32 = c_kv^T . dkv.
 * `status_word` is a device pointer to one 32-bit word (zeroed by the call) that receives the
 * device status; pass it to laga_query_status.
 */
int laga_up_project(const void* c_kv, const void* w_kv_b, int S, int h, int d_c, int d_nope, int d_v,
                    void* kv, void* status_word, void* stream);
int laga_kv_backward(const void* dkv, const void* c_kv, const void* w_kv_b, int S, int h, int d_c,
                     int d_nope, int d_v, void* dc_kv, float* dw_kv_b, unsigned flags, void* status_word,
                     void* stream);

/*
 * The ABSORBED form of the same forward (Section 3.2, baseline B2), for comparison with laga_fwd: the
 * paper's point is what this form costs in training.  Same inputs, outputs and meaning as laga_fwd (the two
 * forms are algebraically identical: q_nope . (W_uk^T c) = (W_uk q_nope) . c), different association:
 *   q_abs[s,i,:] = W_uk[i] q_nope[s,i,:]                 (d_c wide: a batched GEMM over the heads)
 *   scores       = softmax_scale * ( q_abs . c_kv^T + q_rope . k_pe^T )     (576-deep, against the latent itself)
 *   o_lat[s,i,:] = softmax(scores) c_kv                  (d_c-wide accumulator per token and head)
 *   out[s,i,:]   = W_uv[i]^T o_lat[s,i,:]                (a second batched GEMM)
 * where W_uk[i] / W_uv[i] are the K / V column blocks of head i in w_kv_b.  No per-head K or V is formed;
 * instead q_abs and o_lat, S*h*d_c bf16 elements each, live in `workspace` (laga_absorbed_fwd_workspace_bytes):
 * at S=16384, h=16 that is 537 MB against the 134 MB of laga_fwd.  The attention kernel splits the 512
 * latent columns over two CTAs and computes the scores in both, so it executes 3328 FLOP per (query, key)
 * pair (2176 nominal for this form, 640 for the explicit form).  Forward only.
 * Errors and conventions as laga_fwd; `flags` must be 0.
 */
size_t laga_absorbed_fwd_workspace_bytes(int S, int h, int d_c, int d_nope, int d_rope, int d_v);
int laga_absorbed_fwd(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, int S, int h, int d_c,
                      int d_nope, int d_rope, int d_v, float softmax_scale, int causal, void* out, float* lse,
                      void* workspace, size_t workspace_bytes, unsigned flags, void* stream);

/*
 * laga_fwd for callers that have no scratch to give.  (The paper has no counterpart: this is a
 * packaging convenience of the library, not a step of the method.)
 *
 * Who it is for: code that must run the forward but is not in a position to obtain device memory --
 * a plug-in or callback invoked where allocation calls are forbidden, a component of a process whose
 * device memory is entirely owned by someone else's pool, or a latency-sensitive loop that cannot
 * afford cudaMalloc's device-wide synchronisation.  Such a caller still owns its inputs and outputs
 * (same shapes, dtypes, alignment and meaning as laga_fwd) but passes no workspace: the bf16
 * up-projection KV and the launch status word go into a fixed array inside the library image.
 *
 * Limits and rules
 *   - The array holds 16 MiB of KV: S * h <= 32768 (e.g. S=2048 with h=16).  A larger problem returns
 *     LAGA_ERR_WORKSPACE_TOO_SMALL and nothing is enqueued; use laga_fwd with your own workspace.
 *     Every GPU on which the library is loaded carries these 16 MiB (+1 KiB) until the process exits.
 *   - The call allocates and frees nothing (no cudaMalloc/cudaFree, no allocating library routine).
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current) and caches it; make that first call outside any stream capture.  Under CUDA's
 *     lazy module loading the first library call on a device also loads the library's device code, which
 *     is when the array itself comes into being (an implicit device allocation and synchronisation made
 *     by the CUDA runtime, once): keep that first call in the initialisation phase of the program.
 *   - All calls on a device share the one array, and it keeps the previous call's contents.  The
 *     call itself clears the status word and overwrites the KV rows it uses, so back-to-back calls
 *     on ONE stream are safe; calls that can overlap on the GPU (different streams, no ordering
 *     between them) race on it and must be serialised by the caller.
 *   - There is no way to read the device status word of this variant: a bounded device wait that
 *     gives up leaves the outputs incomplete without a report.  Callers that need the report use
 *     laga_fwd + laga_query_status.
 * Errors: as laga_fwd (LAGA_ERR_INVALID_ARG, LAGA_ERR_UNSUPPORTED, LAGA_ERR_CUDA), plus the size
 * limit above.
 */
int laga_fwd_builtin_scratch(const void* q, const void* c_kv, const void* k_pe, const void* w_kv_b, int S,
                             int h, int d_c, int d_nope, int d_rope, int d_v, float softmax_scale, int causal,
                             void* out, float* lse, void* stream);

/*
 * Self-test of the failure-detection path.  Every device-side wait in this library is bounded: a
 * wait that outlives its budget records where it gave up in the status word and the kernel unwinds
 * instead of hanging.  This call launches a one-CTA kernel whose waits can never be satisfied, with a
 * budget of `budget_us` microseconds (1 .. 1000000); afterwards laga_query_status(status_word, ...)
 * returns LAGA_ERR_DEVICE_TIMEOUT with detail 0x54007e57, and the context stays usable.  Nothing
 * faults, traps or spins past the budget.  The paper has no counterpart.
 */
int laga_selftest_bounded_wait(void* status_word, unsigned budget_us, void* stream);

/*
 * Measurement aid.  Registers n_pairs CUDA events pairs (cudaEvent_t passed as void*, created by the
 * caller with timing enabled) that the library records on the launch stream immediately before and
 * after every launch of one kernel, cycling through the pairs launch after launch; n_pairs = 0 stops
 * it.  The caller reads the times (cudaEventElapsedTime) after synchronising, and keeps the events
 * alive while registered.  Intended for benchmarks.  The paper has no counterpart.
 */
#define LAGA_KERNEL_UP_PROJECT 0    /* step 4 GEMM (also the recomputation in laga_bwd)        */
#define LAGA_KERNEL_ATTN_FWD 1      /* step 5 forward attention                               */
#define LAGA_KERNEL_BWD_DELTA 2     /* delta = rowsum(dO * O) and transposed statistics        */
#define LAGA_KERNEL_ATTN_BWD_DKV 3  /* backward attention: dK, dV                              */
#define LAGA_KERNEL_ATTN_BWD_DQ 4   /* backward attention: dQ                                  */
#define LAGA_KERNEL_DKPE_REDUCE 5   /* dk_pe: bf16 rounding of the head-summed rope-column sums */
#define LAGA_KERNEL_DCKV_GEMM 6     /* dc_kv = dKV . W^T                                       */
#define LAGA_KERNEL_DW_GEMM 7       /* dW = c_kv^T . dKV                                       */
#define LAGA_KERNEL_Q_ABSORB 8      /* absorbed form: q_abs = W_uk q_nope (batched over heads)   */
#define LAGA_KERNEL_ATTN_ABSORBED 9 /* absorbed form: latent-space attention                     */
#define LAGA_KERNEL_V_PROJECT 10    /* absorbed form: out = W_uv o_lat (batched over heads)      */
#define LAGA_KERNEL_ATTN_BWD_FUSED 11 /* backward attention in one pass on CTA pairs: dK, dV, dQ sums */
#define LAGA_KERNEL_DQ_CONVERT 12   /* dQ: scale and bf16 rounding of the fp32 sums              */
#define LAGA_KERNEL_COUNT 13
int laga_profile_kernel(int kernel_id, void* const* start_events, void* const* stop_events, int n_pairs);

/*
 * Measurement aid.  The three attention kernels stamp the SM cycle counter and the nanosecond timer when
 * their first CTA starts and when it ends (they are persistent: that CTA lives as long as the kernel) into
 * the workspace's status slot.  This call synchronises `stream`, reads the stamps the last call on
 * `workspace` left and fills two arrays of LAGA_KERNEL_COUNT doubles: the SM clock in MHz the kernel
 * actually ran at (cycles / time) and its duration in milliseconds; entries of kernels without stamps
 * (the GEMMs and the small kernels, or an attention kernel that has not run on this workspace) are 0.
 * Under a power cap this is the clock the tensor pipe really saw, which a coarse host-side sampler
 * cannot resolve for millisecond kernels.  The paper has no counterpart.
 */
int laga_query_kernel_clocks(const void* workspace, void* stream, double* sm_mhz, double* kernel_ms);

/*
 * Synchronises `stream`, reads the status word at the start of `workspace` (or a `status_word`
 * given to a step entry point) and returns LAGA_OK, LAGA_ERR_DEVICE_TIMEOUT, LAGA_ERR_DEVICE_CHECK or
 * LAGA_ERR_CUDA.
 * If `detail` is not NULL it receives the raw device word (which wait gave up).
 */
int laga_query_status(const void* workspace, void* stream, unsigned* detail);

#ifdef __cplusplus
}
#endif
#endif /* LAGA_H_ */

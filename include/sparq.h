/*
 * sparq.h -- C ABI of the B200 (sm_100a) SparQ decode-attention library.
 *
 * SparQ Attention (arXiv 2312.04985) replaces the dense single-token decode attention
 *     y = softmax(q K^T / sqrt(d_h)) V                                   (Eq. (2))
 * by three steps per query head (Section 4):
 *   Step 1  i1 = the r largest components of |q|; approximate scores
 *           s_hat = softmax(q[i1] K[:, i1]^T / tau),  tau = sqrt(d_h ||q[i1]||_1 / ||q||_1)
 *                                                                         (Eqs. (7), (9))
 *   Step 2  i2 = the k positions with the largest s_hat; exact attention over them
 *           y3 = softmax(q K[i2]^T / sqrt(d_h)) V[i2]                      (Eq. (8))
 *   Step 3  alpha = sum of s_hat over i2;  y = alpha y3 + (1 - alpha) v_bar (Eq. (10))
 * with v_bar the running mean of the cached value vectors (Section 3, "Mean value
 * reallocation").  K is stored twice (Section 6): K, position-major [S, d_h], for the row
 * gather of Step 2, and Kt, component-major [d_h, S], for the component gather of Step 1.
 *
 * Conventions common to every call
 *   - fp16 tensors are passed as `const sparq_half*` (IEEE binary16 bit patterns).
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller.
 *     The library allocates no device memory and keeps no pointer after the call returns.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and return without synchronising, except the *_host entry points.
 *   - Layouts (row-major, innermost last):
 *         q, out        [B, Hq, d]
 *         K, V          [B, Hkv, S_max, d]
 *         Kt            [B, Hkv, d, S_max]     with zeros from position seq_lens[b] to the end of
 *                                              its 16-byte vector (8 positions); sparq_cache_build
 *                                              and sparq_cache_append keep it so.  Readers take
 *                                              whole vectors unmasked; finite junk there only
 *                                              loosens an error bound, non-finite junk is unsupported
 *         vsum (fp32), vbar (fp16), k_new, v_new   [B, Hkv, d]
 *         seq_lens (int32)   [B]     number of valid positions of sequence b
 *     Query head h reads KV head h / (Hq / Hkv): consecutive query heads share a KV head
 *     (Section 4, "Grouped query attention").  Each query head selects its own i1 and i2.
 *   - Every fp16 / fp32 tensor pointer and every workspace must be 16-byte aligned (the kernels use
 *     128-bit accesses); a pointer that is not is refused with SPARQ_ERR_ALIGNMENT on the host.
 *   - Supported shapes: d == 128; Hq a multiple of Hkv; S_max a multiple of 8 (rows of Kt
 *     are then 16-byte aligned); 1 <= r <= d; 0 <= k <= SPARQ_K_MAX.
 *   - Return value: SPARQ_OK, or a SPARQ_ERR_* code for anything the host can see; in that
 *     case nothing was launched.  Conditions only the device can see (a bad seq_lens[b], an
 *     append into a full cache) never trap: the kernel raises `*status` (device int32,
 *     may be NULL) to a SPARQ_DEV_* code with atomicMax, writes a defined result for that
 *     sequence (zeros / no write) and carries on.  The caller zeroes `*status` and reads it
 *     whenever it wants to check.
 *   - Non-finite cache values are not supported (no fault; the result is unspecified).
 */
#ifndef SPARQ_H
#define SPARQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t sparq_half;

#define SPARQ_K_MAX 1024
#define SPARQ_HEAD_DIM 128
#define SPARQ_S_MAX_WORKSPACE 262144   /* largest S_max of sparq_decode with a workspace, and of sparq_decode_grouped */
#define SPARQ_G_MAX 8           /* largest group (query heads per KV head) of sparq_decode_grouped */
#define SPARQ_STATIC_SCRATCH_BYTES (8u << 20)   /* scratch built into the library for dense_decode_static */

enum {
    SPARQ_OK = 0,
    SPARQ_ERR_NULL_POINTER = 1,  /* a required pointer is NULL                                   */
    SPARQ_ERR_BAD_SHAPE = 2,     /* B, Hq, Hkv, d or S_max outside the supported shapes          */
    SPARQ_ERR_BAD_RK = 3,        /* r or k out of range                                          */
    SPARQ_ERR_WORKSPACE = 4,     /* workspace NULL or smaller than *_workspace_bytes()           */
    SPARQ_ERR_TOO_LONG = 5,      /* S_max exceeds sparq_max_seq_len() (or, with a workspace,
                                    SPARQ_S_MAX_WORKSPACE)                                      */
    SPARQ_ERR_CUDA = 6,          /* the CUDA runtime refused a launch or a copy                  */
    SPARQ_ERR_STATIC_SCRATCH = 7,/* the problem needs more scratch than the library's fixed
                                    SPARQ_STATIC_SCRATCH_BYTES: use the call that takes a workspace */
    SPARQ_ERR_ALIGNMENT = 8,     /* a tensor or workspace pointer is not 16-byte aligned         */
    SPARQ_ERR_BAD_OPTION = 9,    /* sparq_decode_opt: unknown temperature or window out of range */
    SPARQ_DEV_BAD_SEQ_LEN = 16,  /* device: seq_lens[b] < 1 or > S_max; that out row is zero     */
    SPARQ_DEV_CACHE_FULL = 17,   /* device: append with seq_lens[b] == S_max; nothing written    */
    SPARQ_DEV_TIMEOUT = 18       /* device: an asynchronous copy did not land within the bounded wait;
                                    that out row is zero                                        */
};

/* Human-readable name of a status code (static string, never NULL). */
const char* sparq_status_string(int code);

/* Largest S_max sparq_decode accepts WITHOUT a workspace on the current device (the approximate
 * scores of a unit then live in shared memory, 4 bytes per position).  With the workspace
 * sparq_workspace_bytes() names, the scores go through it instead and the limit is
 * SPARQ_S_MAX_WORKSPACE (only two bitmaps of S_max bits each stay in shared memory). */
int sparq_max_seq_len(void);

/*
 * sparq_cache_build -- derive the SparQ-specific cache state from a prefilled K, V:
 * Kt[b,h,:,t] = K[b,h,t,:] for t < seq_lens[b] (Section 6, "store K twice"), the fp32
 * running sum vsum = sum_{t<n} V[b,h,t,:] and vbar = fp16(vsum / n) (Section 3, v_bar).
 * Kt gets zeros from position seq_lens[b] to the end of its 16-byte vector (the layout's
 * invariant); positions beyond that are left untouched.  seq_lens[b] == 0 gives vsum = vbar = 0.
 */
int sparq_cache_build(const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                      sparq_half* Kt, float* vsum, sparq_half* vbar,
                      int B, int Hkv, int d, int S_max, int32_t* status, void* stream);

/*
 * sparq_cache_append -- one generation step's cache update (Section 3, text around Eq. (3);
 * Appendix "Storing K twice").  For every sequence b, with n = seq_lens[b] read at entry, every
 * KV head writes k_new to K[b,h,n,:] and to Kt[b,h,:,n], v_new to V[b,h,n,:], adds v_new to
 * vsum and refreshes vbar = fp16(vsum / (n + 1)); then seq_lens[b] becomes n + 1.  A decode
 * enqueued after the append on the same stream attends to the new token.
 * n == S_max: nothing is written for b, seq_lens[b] is unchanged, *status = SPARQ_DEV_CACHE_FULL.
 */
int sparq_cache_append(const sparq_half* k_new, const sparq_half* v_new,
                       sparq_half* K, sparq_half* Kt, sparq_half* V, float* vsum, sparq_half* vbar,
                       int32_t* seq_lens, int B, int Hkv, int d, int S_max, int32_t* status, void* stream);

/*
 * sparq_decode -- the SparQ attention step (Section 4, Steps 1-3) for every (b, query head).
 * With n = seq_lens[b] and k_eff = min(k, n):
 *   i1 (r components, ties in |q| to the smaller index), tau (Eq. (9); an all-zero q uses tau = 1),
 *   l_hat[t] = sum_{j in i1} q_j K[t,j] / tau for t < n (Eq. (7)): exact fp16 products summed in
 *   fp32, with every position whose sum lies within the rounding-error bound of the selection
 *   threshold re-decided by its fp64 sum, so that i2 is the set the fp64 definition selects,
 *   i2 = the k_eff largest l_hat (ties to the smaller position), alpha = sum_{t in i2} s_hat[t],
 *   y3 = softmax(q K[i2]^T / sqrt(d)) V[i2] in fp32 (Eq. (8)), out = alpha y3 + (1-alpha) vbar
 *   rounded to fp16 (Eq. (10)).  k == 0 gives out = vbar.
 * Optional outputs (each may be NULL): idx_r [B,Hq,r] int32 = i1 ascending; idx_k [B,Hq,k]
 * int32 = i2 ascending, unused tail -1; alpha [B,Hq] fp32.
 * workspace: optional device scratch; sparq_workspace_bytes() says how much helps for the given
 * shapes (0: none -- a handful of units, or few units per SM on a long cache, run on a kernel
 * that keeps a unit's approximate scores in shared memory).  Three uses, the selected sets
 * identical in all plans (alpha and out may differ in their last bits, the softmax denominator
 * being summed in another order): a cache beyond sparq_max_seq_len() -- the approximate scores
 * of a unit pass through the workspace (4 bytes per position), and with few units every sequence
 * is cut into slices handled by different thread blocks; more units than SMs on the persistent
 * kernel -- 64 bytes for a counter from which the thread blocks draw their units, which evens
 * out their finishing times; four or more units per SM on a cache of about 6,500 to 17,800
 * positions -- the persistent kernel keeps only the upper halves of the scores' sort keys in
 * shared memory and parks the lower halves here (SMs x 3 x 2 bytes per position).  With
 * workspace NULL or too small a plan without scratch is used.  The call clears what it needs;
 * contents are undefined afterwards.
 */
int sparq_decode(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                 const sparq_half* vbar, const int32_t* seq_lens,
                 int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                 sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                 void* workspace, size_t workspace_bytes, int32_t* status, void* stream);
size_t sparq_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max, int r, int k);

/*
 * sparq_decode_opt -- sparq_decode with the settings the paper varies around the algorithm
 * (Section 5.3, "Approximate softmax temperature"; appendix, hyper-parameter table).  Same
 * tensors, outputs, workspace (sparq_workspace_bytes()) and kernels as sparq_decode, which is
 * this call with tau_mode = SPARQ_TAU_L1, realloc = 1, window = 0.
 *   tau_mode  temperature of the approximate softmax of Eq. (7): SPARQ_TAU_L1 = Eq. (9),
 *             SPARQ_TAU_SQRT_D = sqrt(d), SPARQ_TAU_SQRT_R = sqrt(r).  i1 and i2 do not depend
 *             on it (the order of the approximate scores is the same); alpha does.
 *   realloc   0: Step 3 is left out, out = y3 of Eq. (8) (the ablation's setting without
 *             reallocation to the mean value); alpha is still written as Eq. (10) defines it.
 *   window    local window l, 0 <= l <= SPARQ_K_MAX: the l_eff = min(l, k_eff) most recent
 *             positions n - l_eff .. n - 1 always belong to i2, inside the budget of k, and the
 *             other k_eff - l_eff places go to the largest approximate scores among the older
 *             positions (ties to the smaller position); alpha sums s_hat over all of i2.  The
 *             paper lists l = k/4 among SparQ's settings without describing the mechanism: this
 *             is this library's reading of it.
 * Returns SPARQ_ERR_BAD_OPTION for another tau_mode or window, before anything is launched.
 */
enum { SPARQ_TAU_L1 = 0, SPARQ_TAU_SQRT_D = 1, SPARQ_TAU_SQRT_R = 2 };
int sparq_decode_opt(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                     const sparq_half* vbar, const int32_t* seq_lens,
                     int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                     int tau_mode, int realloc, int window,
                     sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                     void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * dense_decode -- dense decode attention, Eq. (2), over the n = seq_lens[b] valid positions:
 * the comparison kernel for the speed-up figure (Section 6.1, "Dense" baseline).  One pass
 * over K and V per KV head serves all Hq/Hkv query heads of its group (eight, four, two or one
 * at a time; eight and four on the tensor cores, the softmax weights rounded to fp16 for the
 * second product).  The sequence is split
 * across thread blocks; partial softmax states go through `workspace`
 * (dense_workspace_bytes(); contents undefined afterwards).
 */
int dense_decode(const sparq_half* q, const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                 int B, int Hq, int Hkv, int d, int S_max, sparq_half* out,
                 void* workspace, size_t workspace_bytes, int32_t* status, void* stream);
size_t dense_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max);

/*
 * dense_decode_static -- dense_decode for callers that must not allocate.  (The paper has no
 * counterpart; this entry point exists for integration only.)
 *
 * Who needs it: a decode step that runs inside a host process whose device memory is owned by
 * someone else -- an inference server that hands its plug-ins fixed buffers and forbids them to call
 * the allocator, or a latency-critical loop in which an allocation (which may synchronise the whole
 * device) is not acceptable.  Such a caller cannot create the `workspace` that dense_decode asks
 * for, so here the scratch for the per-split softmax states is a fixed array of
 * SPARQ_STATIC_SCRATCH_BYTES (8 MiB) inside the library's own device image.  The call allocates
 * and frees nothing, on the host API or through any library; q, K, V, seq_lens, out (and status)
 * are still the caller's buffers, with the same meaning, layout and results as in dense_decode.
 *
 * Limits and rules:
 *   - A problem whose dense_workspace_bytes() exceeds SPARQ_STATIC_SCRATCH_BYTES is refused with
 *     SPARQ_ERR_STATIC_SCRATCH before anything is launched (use dense_decode with a workspace).
 *   - The first call on each device looks up the array's device address (a runtime query, not an
 *     allocation).  Make that first call during set-up, with the device current, and before any
 *     stream capture is started on that device.
 *   - Every GPU that loads the library holds the 8 MiB until the process exits, and all calls on a
 *     device share it.  The array keeps whatever the previous call left; nothing in it needs to be
 *     zero, because every slot that is read was written earlier in the same call.  Two calls that
 *     can overlap on the GPU (different streams, or different host threads) race on it: order
 *     them on one stream or with events.
 */
int dense_decode_static(const sparq_half* q, const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                        int B, int Hq, int Hkv, int d, int S_max, sparq_half* out, int32_t* status, void* stream);

/*
 * sparq_decode_grouped -- the grouped-query variant of the step (Section 4, "Grouped query
 * attention"): the g = Hq / Hkv query heads of a KV head (heads hkv*g .. hkv*g + g - 1) select
 * together.  i1 [B,Hkv,r] = the r components with the largest sum over the group of |q| (ties to
 * the smaller index; the sums are exact); tau (Eq. (9)), l_hat and s_hat (Eq. (7)) per query
 * head over that shared i1; i2 [B,Hkv,k] = the k_eff positions with the largest sum over the
 * group of s_hat (equal sums to the smaller position); per head alpha = its own s_hat mass on
 * i2, y3 = softmax(q K[i2]^T / sqrt(d)) V[i2] (Eq. (8)), and out = alpha y3 + (1 - alpha) vbar
 * (Eq. (10)) when realloc != 0, out = y3 when realloc == 0 (the paper left Step 3 out for its
 * grouped-query models).  The summed scores are evaluated in fp32 (about 1e-5 relative), so two
 * positions whose sums differ by less than that may be selected the other way round than a
 * float64 evaluation would.  g must be 1, 2, 4 or 8.  The r rows of Kt are streamed once per KV
 * head instead of once per query head.
 * workspace: required, sparq_grouped_workspace_bytes() bytes ((g + 1) * 4 bytes per position
 * and KV head); contents undefined afterwards.  Optional outputs as in sparq_decode, with idx_r
 * and idx_k per KV head.  Same error model as sparq_decode.
 */
int sparq_decode_grouped(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                         const sparq_half* vbar, const int32_t* seq_lens,
                         int B, int Hq, int Hkv, int d, int S_max, int r, int k, int realloc,
                         sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                         void* workspace, size_t workspace_bytes, int32_t* status, void* stream);
size_t sparq_grouped_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max);

/*
 * sparq_decode_grouped_opt -- sparq_decode_grouped with the settings of sparq_decode_opt:
 * tau_mode picks every head's temperature (here it can change i2 as well: the summed scores
 * weigh the heads' logits through their softmax), realloc = 0 leaves Step 3 out, and the
 * l_eff = min(window, k_eff) most recent positions always belong to the group's i2, the other
 * places going to the largest summed scores among the older positions.  sparq_decode_grouped is
 * this call with SPARQ_TAU_L1 and window = 0.  SPARQ_ERR_BAD_OPTION as for sparq_decode_opt.
 */
int sparq_decode_grouped_opt(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                             const sparq_half* vbar, const int32_t* seq_lens,
                             int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                             int tau_mode, int realloc, int window,
                             sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                             void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/*
 * sparq_decode_1xk -- sparq_decode for a cache that stores K once (no transposed copy Kt): the
 * variant the paper measures beside the K-stored-twice one (Section 6.1) and leaves open because
 * of the 50 % extra memory Kt costs.  Stage a2 reads whole rows of K (the r selected components
 * of a row are spread over all its 32-byte sectors, so the step moves d/r times the bytes of the
 * Kt stream); results are those of sparq_decode (same selected sets; alpha and out to the last
 * bits).  workspace: required, sparq_1xk_workspace_bytes() bytes; contents undefined afterwards.
 */
int sparq_decode_1xk(const sparq_half* q, const sparq_half* K, const sparq_half* V, const sparq_half* vbar,
                     const int32_t* seq_lens, int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                     sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                     void* workspace, size_t workspace_bytes, int32_t* status, void* stream);
size_t sparq_1xk_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max);

/*
 * sparq_step_host -- one whole generation step driven from HOST buffers: copies q_host
 * [B,Hq,d], k_new_host and v_new_host [B,Hkv,d] (fp16, ideally pinned) to the device, runs
 * sparq_cache_append then sparq_decode on `stream`, copies the result to out_host [B,Hq,d]
 * and waits for the stream.  With k_new_host and v_new_host both NULL, q_host is one buffer
 * that holds q, k_new and v_new back to back (in that order), and they travel in one copy
 * instead of three.  The cache (K, Kt, V, vsum, vbar, seq_lens) stays resident on the
 * device.  staging: device scratch of at least sparq_step_host_staging_bytes() bytes (device
 * copies of the four host tensors, then the workspace sparq_workspace_bytes() names for these
 * shapes, at least 64 bytes).
 */
int sparq_step_host(const sparq_half* q_host, const sparq_half* k_new_host, const sparq_half* v_new_host,
                    sparq_half* K, sparq_half* Kt, sparq_half* V, float* vsum, sparq_half* vbar,
                    int32_t* seq_lens, int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                    sparq_half* out_host, void* staging, size_t staging_bytes, int32_t* status, void* stream);
size_t sparq_step_host_staging_bytes(int B, int Hq, int Hkv, int d, int S_max, int r, int k);

#ifdef __cplusplus
}
#endif
#endif /* SPARQ_H */

/*
 * bebop.h -- C ABI of the speculative rejection-sampling verify step
 * (MTP draft-then-verify rollouts; "Breaking Entropy Bounds: Accelerating RL
 * Training via MTP with Rejection Sampling", Sec. 2.2 and App. G.1).
 *
 * Conventions shared by every entry point
 *   - Every tensor pointer, `workspace` included, is a DEVICE pointer owned by
 *     the caller; scalars are passed by value.  The library never allocates,
 *     frees or synchronises: work is enqueued on `cuda_stream` (a cudaStream_t
 *     passed as void*, NULL = the legacy default stream) and outputs are valid
 *     once that stream reaches the end of the call.
 *   - Logits are row-major with the vocabulary contiguous.  `ld_*` is the
 *     distance between consecutive rows in ELEMENTS (>= V).  Row (b,k) of a
 *     [B,R,V] tensor starts at element (b*R + k) * ld.  The base pointer and
 *     ld * sizeof(element) must be multiples of 16 bytes.
 *   - -inf logits are legal (masked vocabulary, probability 0).
 *   - Errors that can be seen on the host (NULL required pointer, B/K/V out of
 *     range, K > BEBOP_MAX_K, ld < V, misalignment, workspace too small,
 *     temperature_all <= 0 with no per-row tensor, device not sm_100) return a
 *     status BEFORE any launch and write nothing.
 *   - Data-dependent anomalies never trap; they set bits in row_status[b] and
 *     the row still yields a defined result (see BEBOP_ROW_*).  A row with any
 *     of the FATAL bits yields accept_len = 0, out_tokens = -1, tv = 0.
 *   - Calls sharing one workspace must not overlap on the GPU.
 */
#ifndef BEBOP_H_
#define BEBOP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BEBOP_MAX_K 32   /* accept bits of one sequence fit one warp ballot */

typedef enum {
    BEBOP_OK = 0,
    BEBOP_ERR_NULL = 1,
    BEBOP_ERR_SHAPE = 2,
    BEBOP_ERR_DTYPE = 3,
    BEBOP_ERR_ALIGN = 4,
    BEBOP_ERR_WORKSPACE = 5,
    BEBOP_ERR_TEMPERATURE = 6,
    BEBOP_ERR_ARCH = 7,
    BEBOP_ERR_CUDA = 8,
    BEBOP_ERR_STATIC_SCRATCH = 9
} bebop_status_t;

typedef enum { BEBOP_F32 = 0, BEBOP_BF16 = 1 } bebop_dtype_t;

/* bits of row_status[b] */
#define BEBOP_ROW_NONFINITE 1   /* NaN or +inf logit in a row the method reads (FATAL)   */
#define BEBOP_ROW_EMPTY 2       /* a row whose logits are all -inf (FATAL)                */
#define BEBOP_ROW_BAD_TOKEN 4   /* draft token id outside [0,V) (FATAL)                   */
#define BEBOP_ROW_ZERO_RESID 8  /* residual mass 0 at a rejected position: drew from p    */
#define BEBOP_ROW_BAD_TEMP 16   /* per-row temperature <= 0 or non-finite (FATAL)         */
#define BEBOP_ROW_WAIT_EXPIRED 32 /* a bounded device-side wait gave up (result undefined) */
#define BEBOP_ROW_FATAL (1 | 2 | 4 | 16)

/* Bytes of device scratch the three entry points below need for this shape
 * (pure host function; 0 on invalid arguments).  bebop_verify and
 * bebop_greedy_verify of shape (B,K,V) use bebop_workspace_bytes(B,K,V,dt);
 * bebop_tv of N rows uses bebop_workspace_bytes(N,1,V,dt).  The buffer must be
 * 256-byte aligned; its contents need not be initialised. */
size_t bebop_workspace_bytes(int B, int K, int V, bebop_dtype_t dt);

/*
 * Chain rejection-sampling verification (App. G.1, Algorithm 3), with logits in
 * place of cached probabilities and the uniforms supplied by the caller.
 * For each sequence b with L = draft_len[b] drafts and temperature tau_b:
 *   p_k = softmax(target[b,k,:]/tau_b), q_k = softmax(draft[b,k,:]/tau_b)   (Sec. 2.2)
 *   accept x_k while u_accept[b,k] * q_k(x_k) < p_k(x_k); stop at the first reject
 *   at a reject at position n: draw y from max(0, p_n - q_n)/Z by inverse CDF,
 *     y = min{ v : sum_{v'<=v} r(v') >= u_final[b] * Z }
 *   if all L accepted: draw the bonus token the same way from p_L (target row L)
 *   tv[b,k] = sum_v max(0, p_k - q_k) = d_TV(p_k, q_k) = 1 - E[accept]   (Eq. reject_sample)
 * Rows k >= L are never read; the bonus row is read only when all L are accepted.
 * The draw agrees with an fp64 evaluation of the definition except on near-ties:
 * an fp32 prefix sum decides the token only where the crossing clears its error
 * bound on both sides; the remaining sequences are re-drawn in double precision.
 *
 * target_logits [B,K+1,V], draft_logits [B,K,V] : dtype dt
 * draft_tokens  [B,K] int32; draft_len [B] int32 in 0..K, or NULL (= K)
 * temperature   [B] fp32, or NULL -> temperature_all (> 0) for every row
 * u_accept [B,K], u_final [B] : fp32 uniforms in the open interval (0,1)
 * accept_len [B], out_tokens [B,K+1] (x_1..x_n, y, then -1) : int32 outputs
 * tv, p_draft, q_draft [B,K] fp32 outputs, each may be NULL (0 beyond draft_len).  With tv = NULL the
 *   residuals are formed only at the position a token is drawn from, and the call reads that much less.
 * row_status [B] int32 output, may be NULL
 */
bebop_status_t bebop_verify(
    const void* target_logits, int64_t ld_target,
    const void* draft_logits, int64_t ld_draft,
    const int32_t* draft_tokens, const int32_t* draft_len,
    const float* temperature, float temperature_all,
    const float* u_accept, const float* u_final,
    int B, int K, int V, bebop_dtype_t dt,
    int32_t* accept_len, int32_t* out_tokens,
    float* tv, float* p_draft, float* q_draft, int32_t* row_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Total-variation distance of N independent row pairs (Eq. reject_sample and
 * the identity of Sec. 3.3; forward value of the TV loss, App. F Algorithm 1):
 *   tv[n]    = sum_v max(0, p - q), clamped to [0,1]
 *   s_aux[n] = sum_v q(v) * 1[q(v) <= p(v)]   (the scalar S of Eq. tv_grad), may be NULL
 * with p = softmax(target[n,:]/tau_n), q = softmax(draft[n,:]/tau_n).
 * target_logits, draft_logits [N,V]; temperature [N] or NULL; row_status [N] or NULL.
 */
bebop_status_t bebop_tv(
    const void* target_logits, int64_t ld_target,
    const void* draft_logits, int64_t ld_draft,
    const float* temperature, float temperature_all,
    int N, int V, bebop_dtype_t dt,
    float* tv, float* s_aux, int32_t* row_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * bebop_tv without a workspace argument (a convenience of this library; the paper has no
 * counterpart).  Same definition, same outputs (to fp32 rounding: it always runs the split-row kernels,
 * bebop_tv the pipelined kernel where the shape admits it) and same errors as bebop_tv, with the per-slice
 * partials of the sweep kept in a scratch array that is part of the library image
 * (BEBOP_TV_STATIC_SCRATCH_BYTES = 1 MiB, one copy per device).  The call allocates nothing and
 * frees nothing.
 *   - Limit: 16 + 8 bytes per (row pair, slice), in two arrays that each start on a 256-byte boundary, must fit
 *     the array: up to 43,680 (row pair, slice) entries.  Rows are cut into fewer slices as N grows (32 for a
 *     handful of long rows, 1 beyond a few thousand rows), so N up to a few thousand always fits and
 *     N > 43,680 never does.  A shape
 *     that does not fit returns BEBOP_ERR_STATIC_SCRATCH before any launch; use bebop_tv with a
 *     caller workspace then.
 *   - Set-up: the first call on each device looks up the device address of the array
 *     (cudaGetSymbolAddress).  Make that first call before starting a stream capture, not inside
 *     one; later calls only enqueue kernels and can be captured.
 *   - The array is shared by every call on the device: two calls that may overlap on the GPU
 *     (different streams, or graphs replayed concurrently) race on it.  Serialise them, or give
 *     the overlapping call its own workspace through bebop_tv.
 *   - Nothing in the array has to start at zero and nothing is kept between calls.
 */
#define BEBOP_TV_STATIC_SCRATCH_BYTES (1u << 20)
bebop_status_t bebop_tv_static(
    const void* target_logits, int64_t ld_target,
    const void* draft_logits, int64_t ld_draft,
    const float* temperature, float temperature_all,
    int N, int V, bebop_dtype_t dt,
    float* tv, float* s_aux, int32_t* row_status, void* cuda_stream);

/*
 * Greedy-draft mode (the deterministic limit of target-only sampling, Sec. 2.2):
 * g_k = lowest index attaining max_v target[b,k,v]; accept x_k while x_k == g_k;
 * emit g at the stop position (g_L when all L drafts match).  All L+1 target
 * rows of a sequence are read; temperature plays no role.
 */
bebop_status_t bebop_greedy_verify(
    const void* target_logits, int64_t ld_target,
    const int32_t* draft_tokens, const int32_t* draft_len,
    int B, int K, int V, bebop_dtype_t dt,
    int32_t* accept_len, int32_t* out_tokens, int32_t* row_status,
    void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Test and measurement hooks (no counterpart in the paper).  They set process-wide switches that every later
 * call in the process sees: not thread-safe, and not meant for code that serves requests.
 * bebop_debug_force_general_path(mode) chooses the kernels behind bebop_verify, bebop_tv and bebop_greedy_verify:
 * 0 (the default) the faster, by measurement, of the fused and the pipelined kernel for the shape, and the
 * split-row general kernels for shapes neither takes; 1 the general kernels always; 2 never the fused kernel;
 * 3 the fused kernel wherever it applies (the greedy mode has no fused form).  All give the same results up to
 * the documented tolerances.  bebop_debug_last_kernel() says what the last of these calls ran: 1 the general kernels,
 * 2 the pipelined kernel, 3 the fused kernel (0: no call yet).
 * bebop_debug_fallback_offset returns the byte offset, inside the workspace of this
 * shape, of an int32 that after a bebop_verify call holds the number of sequences
 * whose draw was re-done by the fp64 kernels.
 * bebop_debug_set_timing_events(start, stop): two cudaEvent_t handles that the next
 * bebop_verify calls record around the main (pipelined or fused) kernel, on the caller's stream (NULL,
 * NULL switches it off).
 * bebop_debug_expire_wait(which): the next call's device-side wait number `which` (1: the re-draw kernel's wait
 * for the list of sequences; 2: the main kernel's wait for what other CTAs deliver) gives up at once, as if
 * its bound had run out: the call still returns, every row_status carries BEBOP_ROW_WAIT_EXPIRED, and the call
 * after it is normal again (0: off).  For the test of the bounded waits; nothing is trapped or hung.
 * bebop_debug_set_draw_kappa(kappa): the factor in the error bound that decides whether bebop_verify keeps a token
 * drawn from the fp32 prefix sums or re-draws it in double (built-in value 4; a negative argument restores it;
 * 0 keeps every fp32 draw).  For the test that shows how much room the built-in value leaves.
 */
void bebop_debug_force_general_path(int on);
int bebop_debug_last_kernel(void);
size_t bebop_debug_fallback_offset(int B, int K, int V, bebop_dtype_t dt);
void bebop_debug_set_timing_events(void* start, void* stop);
void bebop_debug_expire_wait(int which);
void bebop_debug_set_draw_kappa(float kappa);

/* Static, host-side, human-readable name of a status code. */
const char* bebop_status_string(bebop_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* BEBOP_H_ */

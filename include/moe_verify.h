/*
 * moe_verify.h -- C ABI of the B200 (sm_100a) sparse-MoE FFN layer as run by the target
 * model's speculative-decoding verification step.
 *
 * Verification pushes T = B*(gamma+1) tokens (gamma draft tokens plus one bonus token per
 * sequence, Sec. 3.1) through the target model at once.  In a sparse MoE layer a router
 * activates top_k of n_experts experts per token (Sec. 1; Sec. 3.2, Eq. PrX), only the
 * experts that received a token are executed -- so only their weights are streamed from
 * HBM, the quantity N(t) of Eq. N(t) -- and each activated expert sees on average
 * T_exp tokens (Eq. T_exp).  The entry points below are the steps of that layer.
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, 16-byte aligned, dense
 *     row-major with the innermost extent contiguous.  The library never allocates or
 *     frees device memory; scratch comes from the caller's workspace `ws`.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls only
 *     enqueue work; they never synchronise.  Results are valid once the stream has
 *     reached the end of the call's work.
 *   - bf16 tensors are passed as void*.
 *   - Errors detectable on the host (null / misaligned pointers, bad shapes, workspace
 *     too small) are reported by the return code BEFORE anything is launched.
 *   - Router logits must be finite; otherwise the selection order is unspecified (never
 *     out of bounds).
 *   - The layer is token-wise: B and gamma only fix T.
 *   - Shape limits: 1 <= top_k <= n_experts <= MOE_MAX_EXPERTS, top_k <= MOE_MAX_TOPK,
 *     hidden, inter and shared_inter multiples of 32, T >= 1, T*top_k < 2^24.
 */
#ifndef MOE_VERIFY_H_
#define MOE_VERIFY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOE_MAX_EXPERTS 512
#define MOE_MAX_TOPK 16

typedef enum {
    MOE_OK = 0,
    MOE_ERR_INVALID_ARG = 1, /* null / misaligned pointer, shape outside the limits      */
    MOE_ERR_UNSUPPORTED = 2, /* valid request this build cannot run (e.g. wrong GPU arch) */
    MOE_ERR_WORKSPACE = 3,   /* ws_bytes smaller than moe_workspace_bytes()               */
    MOE_ERR_CUDA = 4,        /* a CUDA runtime call failed (launch error)                 */
    MOE_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (see moe_check)        */
} moe_status_t;

typedef enum { MOE_SCORE_SOFTMAX = 0, MOE_SCORE_SIGMOID = 1 } moe_score_t;

/* Layer shape and router variant.  The paper fixes none of these (it analyses stock
 * models); they are the knobs of the model families it measures (Sec. 4). */
typedef struct {
    int32_t hidden;       /* H                                                            */
    int32_t n_experts;    /* E  routed experts                                            */
    int32_t top_k;        /* K  experts activated per token (Sec. 3.2)                    */
    int32_t inter;        /* I  routed-expert intermediate size                           */
    int32_t shared_inter; /* I_s shared-expert intermediate size, 0 = no shared expert    */
    int32_t score_fn;     /* moe_score_t: softmax over all E logits, or per-expert sigmoid */
    int32_t renormalize;  /* 1: the K selected scores are divided by their sum            */
    int32_t shared_gate;  /* 1: shared expert scaled by sigmoid(x . w_shared_gate)        */
    float routed_scale;   /* multiplies the K gate weights (1.0 in every benchmark shape) */
} moe_config_t;

typedef struct {
    const float *w_router;     /* [E, H] fp32                                             */
    const float *router_bias;  /* [E] fp32 added to the logits, or NULL                   */
    const void *w_gate;        /* [E, I, H] bf16                                          */
    const void *w_up;          /* [E, I, H] bf16                                          */
    const void *w_down;        /* [E, H, I] bf16                                          */
    const void *ws_gate;       /* [I_s, H] bf16 (shared expert) or NULL                   */
    const void *ws_up;         /* [I_s, H] bf16 or NULL                                   */
    const void *ws_down;       /* [H, I_s] bf16 or NULL                                   */
    const void *w_shared_gate; /* [H] bf16, needed when shared_gate = 1                   */
} moe_weights_t;

/* Optional copies of the layer's intermediates (any member may be NULL). */
typedef struct {
    float *logits;     /* [T, E]   */
    int32_t *topk_idx; /* [T, K]   */
    float *topk_w;     /* [T, K]   */
    int32_t *counts;   /* [E]      */
    int32_t *offsets;  /* [E+1]    */
    int32_t *perm;     /* [T*K]    */
    int32_t *inv_perm; /* [T*K]    */
    int32_t *active;   /* [E]      */
    int32_t *n_active; /* [1]      */
} moe_debug_out_t;

/* Bytes of workspace any entry point needs for up to max_tokens tokens (0 on bad args).
 * The workspace need not be initialised. */
size_t moe_workspace_bytes(const moe_config_t *cfg, int32_t max_tokens);

/* Test aid (no counterpart in the paper): region `index` (0, 1, ...) of the layout a call with T
 * tokens uses inside its workspace, as byte offset and bytes in use.  Regions start 256-byte
 * aligned and are separated by at least 256 bytes that no kernel ever writes, so a caller that
 * fills the workspace with a pattern first can detect a stray store afterwards.  Returns
 * MOE_ERR_INVALID_ARG past the last region. */
moe_status_t moe_workspace_region(const moe_config_t *cfg, int32_t T, int32_t index,
                                  size_t *offset, size_t *bytes);

/* Router logits (the gate of Sec. 1):  logits[t,e] = x[t,:] . w_router[e,:] (+ bias[e]),
 * fp32 accumulation.  If shared_scale != NULL and cfg->shared_gate, also writes
 * shared_scale[t] = sigmoid(x[t,:] . w_shared_gate).
 *   x [T,H] bf16; logits [T,E] fp32 out; shared_scale [T] fp32 out or NULL. */
moe_status_t moe_router_logits(const moe_config_t *cfg, const moe_weights_t *w, const void *x,
                               int32_t T, float *logits, float *shared_scale, void *stream);

/* Top-K routing (Sec. 3.2: each token activates K of E experts).  Selection is on the
 * fp32 logits: slot j holds the expert with the j-th largest logit, equal logits resolve
 * to the lower expert index.  topk_w[t,j] is the softmax-over-all-E (or sigmoid) score of
 * that expert, divided by the sum over the K slots if cfg->renormalize, times
 * cfg->routed_scale.
 *   logits [T,E] fp32; topk_idx [T,K] int32 out; topk_w [T,K] fp32 out. */
moe_status_t moe_route_topk(const moe_config_t *cfg, const float *logits, int32_t T,
                            int32_t *topk_idx, float *topk_w, void *stream);

/* Token-to-expert grouping (Sec. 3.3 (3): after the gate each expert processes only its
 * subset of tokens; experts with no token are never touched).  Assignment a = t*K + j
 * belongs to expert topk_idx[a].  Outputs, all int32:
 *   counts[e]      number of assignments of expert e
 *   offsets[0..E]  exclusive prefix sum of counts, offsets[E] = T*K
 *   perm[i]        assignment at sorted position i; order is (expert, a) ascending (stable)
 *   inv_perm[a]    sorted position of assignment a
 *   active[0..n_active)  ascending ids of experts with counts > 0, remaining entries -1
 *   n_active[0]    the number of activated experts, the measured N(t) of Eq. N(t). */
moe_status_t moe_permute(const moe_config_t *cfg, const int32_t *topk_idx, int32_t T,
                         int32_t *counts, int32_t *offsets, int32_t *perm, int32_t *inv_perm,
                         int32_t *active, int32_t *n_active, void *stream);

/* Expert FFNs over the activated experts only (Sec. 3.3 (2): the cost is loading the N
 * activated experts).  For sorted position i (expert e, token t = perm[i] / K):
 *   y[i,:] = W_down[e] . ( silu(W_gate[e] . x[t,:]) * (W_up[e] . x[t,:]) )
 * bf16 inputs, fp32 accumulation, the SwiGLU intermediate rounded once to bf16.
 * If shared_y != NULL and cfg->shared_inter > 0 the shared expert runs on all T rows in the
 * same launches: shared_y[t,:] = FFN_shared(x[t,:]).
 *   x [T,H] bf16; offsets, perm, active, n_active as written by moe_permute;
 *   y [T*K, H] bf16 out (sorted order); shared_y [T,H] bf16 out or NULL;
 *   ws / ws_bytes: workspace of at least moe_workspace_bytes(cfg, T). */
moe_status_t moe_grouped_swiglu(const moe_config_t *cfg, const moe_weights_t *w, const void *x,
                                int32_t T, const int32_t *offsets, const int32_t *perm,
                                const int32_t *active, const int32_t *n_active, void *y,
                                void *shared_y, void *ws, size_t ws_bytes, void *stream);

/* moe_grouped_swiglu without a caller-provided workspace (the paper has no counterpart; this
 * is a packaging variant of the step above, same kernels, same results).
 *
 * Who needs it: callers that may not allocate device memory at the point where they run the
 * layer -- an inference server that froze its memory plan at start-up, a plugin living inside
 * another framework's allocator, a latency-critical loop that cannot risk the implicit
 * device synchronisation of cudaMalloc/cudaFree -- and therefore cannot size and pass `ws`.
 * The scratch (segment plan and the bf16 SwiGLU intermediates) lives in a fixed array of
 * MOE_STATIC_SCRATCH_BYTES inside the library image; each GPU that loads the library holds it
 * until the process exits.  The call itself allocates nothing, on host or device.
 *
 * Limit: the request must satisfy, with A = T*top_k and every term rounded up to 256 bytes and
 * followed by 256 bytes of guard,
 *   256 + 64 + 52*(n_experts + A/128 + 1) + 4*(T/64 + 1) + 2*A*hidden + 2*A*inter + 2*T*shared_inter
 *     <= MOE_STATIC_SCRATCH_BYTES,
 * otherwise MOE_ERR_WORKSPACE is returned and nothing is launched (use moe_grouped_swiglu).
 *
 * Set-up: the first call on a device looks up the array's device address (once per device,
 * with that device current).  Make that first call outside any stream capture.
 * Sharing: every call on a device uses the same array and leaves its contents behind; the
 * call clears what it needs cleared.  Two calls whose work overlaps on the GPU (different
 * streams, or threads) race on it -- order them on one stream or with events.
 * Arguments, results and host-side error codes otherwise as for moe_grouped_swiglu; the
 * device-side status (a bounded wait that gave up) is read with moe_check_static. */
#define MOE_STATIC_SCRATCH_BYTES (8u << 20)
moe_status_t moe_grouped_swiglu_static(const moe_config_t *cfg, const moe_weights_t *w,
                                       const void *x, int32_t T, const int32_t *offsets,
                                       const int32_t *perm, const int32_t *active,
                                       const int32_t *n_active, void *y, void *shared_y,
                                       void *stream);

/* moe_check for moe_grouped_swiglu_static (no counterpart in the paper): synchronises `stream`
 * and reports the status word inside the library's scratch array of the current device --
 * MOE_OK, MOE_ERR_TIMEOUT (a bounded wait inside a kernel of some static call since the last
 * report gave up; that call's outputs are invalid, the context stays usable), or MOE_ERR_CUDA.
 * The word is shared by every static call on the device and is cleared by this report.
 * Allocates nothing. */
moe_status_t moe_check_static(void *stream);

/* moe_selftest_wait_limit on the status word of the library's scratch array: lets a caller of
 * the static entry point see the failure path end to end (report through moe_check_static,
 * next call unaffected) without anything faulting. */
moe_status_t moe_selftest_wait_limit_static(int32_t limit_us, void *stream);

/* Gate-weighted combine:
 *   out[t,:] = sum_{j<K} topk_w[t,j] * y[inv_perm[t*K+j],:]  (slot order, fp32)
 *            + shared_scale[t] * shared_y[t,:]                (if shared_y != NULL;
 *                                                              scale 1 if shared_scale NULL)
 * rounded once to bf16.  y [T*K,H] bf16; out [T,H] bf16. */
moe_status_t moe_combine(const moe_config_t *cfg, const void *y, const int32_t *inv_perm,
                         const float *topk_w, const void *shared_y, const float *shared_scale,
                         int32_t T, void *out, void *stream);

/* The whole layer for one verification step of B sequences with gamma draft tokens each:
 * T = B*(gamma+1) rows of x go through moe_router_logits, moe_route_topk, moe_permute,
 * moe_grouped_swiglu and moe_combine; the result equals the dense-masked definition
 *   out[t] = sum_e m[t,e] * FFN_e(x[t]) + s[t] * FFN_shared(x[t]).
 * T_T(B,gamma) of Sec. 3.1 is the duration of this call's work.
 *   x, out [T,H] bf16; dbg NULL or pointers that receive copies of the intermediates.
 * Numerics: as the separate steps, except that while the down projection has too few work
 * items to keep every SM streaming (few tokens, or few experts with long reductions) its
 * reduction is cut into up to 8 k chunks whose partial sums are rounded to bf16 before the
 * combine adds them in fp32: an expert output then carries up to 8 bf16 roundings instead of
 * one, the shared expert's likewise (its chunk count depends on the shape only).  How many
 * chunks are used depends on T, so a token's low-order bits may differ between batch sizes;
 * the result stays within the layer's stated tolerance at every size.
 * One to four tokens (with T*top_k <= 32 and a shared expert of moderate size) run as ONE
 * cooperative launch: partial router logits, then top-k and grouping repeated by every CTA,
 * then the expert projections on the CUDA cores with the weights streamed once.  There the
 * SwiGLU intermediate is still rounded to bf16, but the expert outputs stay in fp32 until the
 * gate-weighted sum, which is rounded once.  Calls that use the same workspace must not overlap
 * on the GPU (as for every entry point); the device needs cooperative-launch support, else
 * the call takes the kernel sequence of the larger sizes. */
moe_status_t moe_verify_layer(const moe_config_t *cfg, const moe_weights_t *w, const void *x,
                              int32_t B, int32_t gamma, void *out, const moe_debug_out_t *dbg,
                              void *ws, size_t ws_bytes, void *stream);

/* Synchronises `stream` and returns the device-side status word of the workspace:
 * MOE_OK, MOE_ERR_TIMEOUT if a bounded wait inside a kernel gave up (outputs are then
 * invalid but the context stays usable), or MOE_ERR_CUDA.  The word is sticky: a wait that
 * gave up in ANY call on this workspace since the last report keeps it raised (later calls do
 * not clear it), and this call clears it after reading, so every failure is reported once. */
moe_status_t moe_check(void *ws, void *stream);

/* Self-test of the failure path (no counterpart in the paper).  Every wait inside the kernels is
 * bounded; when one gives up, the kernel raises the workspace's status word and returns, and
 * moe_check reports MOE_ERR_TIMEOUT while the context stays usable.  This call enqueues two tiny
 * kernels that run exactly those waits -- the one the down projection uses for the progress
 * counters of the gate/up pass, then the one the one-launch layer of a few tokens uses for its
 * grid barrier and per-expert counters -- each on a word nothing ever advances, each with a limit
 * of limit_us microseconds (1 .. 1000000).  ws: any workspace of at least 256 bytes; its status
 * word is overwritten (the fourth 32-bit word of ws reads 1 once the second wait has given up).
 * Returns at once; the outcome is read with moe_check(ws, stream). */
moe_status_t moe_selftest_wait_limit(void *ws, int32_t limit_us, void *stream);

/* Measurement aid (no counterpart in the paper; its Sec. 3.3 model attributes the layer's
 * time to weight loading, which the benchmark verifies per kernel).  Every following
 * moe_verify_layer call of this thread records start_event before and stop_event after the
 * kernel of the given stage on the call's stream.  Events are cudaEvent_t passed as void*,
 * created and owned by the caller; stage < 0 switches the recording off.  A stage whose work
 * another stage's kernel does for the call's size (small batches: top-k and gather inside the
 * grouping kernel) records nothing. */
typedef enum {
    MOE_STAGE_ROUTER_LOGITS = 0,
    MOE_STAGE_ROUTE_TOPK = 1,
    MOE_STAGE_PERMUTE = 2,
    MOE_STAGE_PLAN = 3,
    MOE_STAGE_GATE_UP = 4,
    MOE_STAGE_DOWN = 5,
    MOE_STAGE_COMBINE = 6,
    MOE_STAGE_GATHER = 7 /* token rows into sorted order */
} moe_stage_t;
moe_status_t moe_profile_stage(int32_t stage, void *start_event, void *stop_event);

/* Number of kernels the last moe_verify_layer call on this thread enqueued. */
int32_t moe_last_launch_count(void);

const char *moe_status_string(moe_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* MOE_VERIFY_H_ */

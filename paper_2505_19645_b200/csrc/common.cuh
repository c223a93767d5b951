// Shared declarations of the CUDA path: workspace layout, segment plan, device helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "device_once.h"
#include "moe_verify.h"

namespace moe {

// ---------------------------------------------------------------------------------------
// Segment plan.  The token rows of an activated expert (a "group") are cut into segments of
// at most SEG_TOKENS (or, for calls whose groups run to hundreds of rows, 2 * SEG_TOKENS)
// consecutive sorted rows, the N extent of one tensor-core instruction.
// The plan lists one entry per segment; every entry carries its whole group, so that any
// segment index leads to the group, its first segment and its number of segments.  The plan
// is derived from the grouping offsets on the device: the host never needs the
// data-dependent counts and no launch waits for a copy.
// ---------------------------------------------------------------------------------------
constexpr int SEG_TOKENS = 128;
constexpr int PLAN_HEADER_INTS = 16;

// Status region (first of the workspace): word [0] is the device status word, raised by a
// bounded wait that gave up and left alone by everything else until moe_check reads and clears
// it; word [1] holds STATUS_MAGIC once the region has been initialised (a fresh workspace holds
// garbage: the first kernel of every call clears word [0] unless the magic is already there).
constexpr int32_t STATUS_MAGIC = 0x4d6f4553;

struct Segment {
    int32_t expert;     // routed expert id of the group
    int32_t row0;       // first sorted row of the group
    int32_t n;          // rows of the group (all its segments together)
    int32_t first_seg;  // plan index of the group's first segment
};

// plan header (ints): [0] number of segments over all activated experts, [1] the same,
//                     [2], [3] routed work claimed so far by the gate/up and the down pass
// A segment with its group: everything a CTA needs to start on a (segment, tile) item in one
// 32-byte load.
struct __align__(16) PairEntry {
    int32_t expert, row0, n, first_seg;  // the group (as in Segment)
    int32_t seg;                         // plan index of the segment
    int32_t pad[3];
};

struct PlanView {
    int seg_rows;         // token rows per segment: SEG_TOKENS or twice that (set by the host)
    int32_t *header;      // written by the plan; [2], [3] advanced by the FFN kernels
    Segment *seg;         // capacity max_segments()
    PairEntry *pairs;     // one entry per segment (with its group), capacity max_segments()
    // Progress of the gate/up pass, read by the down pass: 16-row units of h written so far
    // (counted once per epilogue warp) for every routed segment [max_segments()] and for
    // every 128-row segment of the shared expert [max_shared_segments()].
    int32_t *done_routed;
    int32_t *done_shared;
};

// (the shared expert's rows may be cut into half segments, see the FFN launchers)
__host__ __device__ inline int max_shared_segments(int T) { return (T + SEG_TOKENS / 2 - 1) / (SEG_TOKENS / 2); }

__host__ __device__ inline int max_segments(int E, int A) { return E + A / SEG_TOKENS + 1; }

// ---------------------------------------------------------------------------------------
// Workspace layout (every region 256-byte aligned).
// ---------------------------------------------------------------------------------------
constexpr int WS_MAX_REGIONS = 32;
constexpr size_t WS_GUARD_BYTES = 256;  // never written: lets a test detect a store that strays

struct Workspace {
    size_t status;        // int32[64]: [0] device status word, [1] STATUS_MAGIC once initialised
    size_t logits;        // f32 [T,E]
    size_t topk_idx;      // i32 [T,K]
    size_t topk_w;        // f32 [T,K]
    size_t shared_scale;  // f32 [T]
    size_t counts;        // i32 [E]
    size_t offsets;       // i32 [E+1]
    size_t active;        // i32 [E]
    size_t n_active;      // i32 [1]
    size_t perm;          // i32 [A]
    size_t inv_perm;      // i32 [A]
    size_t plan_header;   // i32 [PLAN_HEADER_INTS]
    size_t plan_seg;      // Segment[max_segments]
    size_t plan_pairs;    // PairEntry [max_segments]
    size_t plan_done;     // i32 [max_segments + max_shared_segments]
    size_t plan_done_shared_at;  // index of the shared expert's counters inside plan_done
    size_t x_sorted;      // bf16 [A, H]      token rows in sorted order
    size_t h;             // bf16 [A, I]      SwiGLU intermediate, sorted order
    size_t h_shared;      // bf16 [T, I_s]
    size_t y;             // bf16 [A, H]      expert outputs, sorted order
    size_t y_shared;      // bf16 [shared_down_parts, T, H]: partial sums per k chunk
    size_t rl_planes;     // bf16 [3, R, H]: router rows as three bf16 terms (large batches only)
    size_t rl_partial;    // f32 [k chunks, T, R]: partial logits (large batches only)
    size_t small_logit_part;  // unit counters, then f32 [E + 1, column chunks, 4]: partial logits of the one-launch layer
    size_t small_h;           // bf16 [rows, padded I] + [T, padded I_s]: SwiGLU intermediates of the one-launch layer
    size_t total;
    // every region in layout order (offset, bytes in use); the bytes between two regions --
    // the rounding up to 256 and a guard of WS_GUARD_BYTES -- belong to no kernel
    int n_regions;
    size_t region_off[WS_MAX_REGIONS], region_bytes[WS_MAX_REGIONS];
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Carves regions off a running offset: 256-byte aligned starts, a guard behind each.
struct WorkspaceCarver {
    Workspace &w;
    size_t off = 0;
    explicit WorkspaceCarver(Workspace &ws) : w(ws) { w.n_regions = 0; }
    size_t take(size_t bytes)
    {
        const size_t at = off;
        if (w.n_regions < WS_MAX_REGIONS) {
            w.region_off[w.n_regions] = at;
            w.region_bytes[w.n_regions] = bytes;
            ++w.n_regions;
        }
        off = align_up(off + bytes, 256) + WS_GUARD_BYTES;
        return at;
    }
};

// k chunks the shared expert's down projection is split into inside moe_verify_layer (each
// chunk is a work unit of its own and writes a partial [T,H] plane that the combine step sums)
int shared_down_parts(const moe_config_t &c);
// k chunks of the routed groups' down projection for T tokens (1 once the pass has enough
// work items without), and the largest assignment count A' = T' * top_k over T' <= T at which
// the chunks are still used: y must hold ROUTED_SPLIT_MAX_PARTS planes of A' rows.
constexpr int ROUTED_SPLIT_MAX_PARTS = 8;
int routed_down_parts(const moe_config_t &c, int T);
size_t routed_split_max_rows(const moe_config_t &c, int T);

// regions of the tensor-core router-logit path (0 bytes where a call does not use it)
bool router_logits_tc_applies(const moe_config_t &c, int T);
size_t router_tc_plane_bytes(const moe_config_t &c, int T);
size_t router_tc_partial_bytes(const moe_config_t &c, int T);

// the whole layer in one launch for a handful of tokens (layer_small.cu); its two regions
bool layer_small_applies(const moe_config_t &c, int T);
size_t layer_small_logit_part_bytes(const moe_config_t &c);
size_t layer_small_h_bytes(const moe_config_t &c, int T);

inline Workspace workspace_layout(const moe_config_t &c, int T)
{
    Workspace w{};
    const size_t A = (size_t)T * c.top_k, E = c.n_experts, H = c.hidden;
    WorkspaceCarver cut(w);
    w.status = cut.take(64 * 4);
    w.logits = cut.take((size_t)T * E * 4);
    w.topk_idx = cut.take(A * 4);
    w.topk_w = cut.take(A * 4);
    w.shared_scale = cut.take((size_t)T * 4);
    w.counts = cut.take(E * 4);
    w.offsets = cut.take((E + 1) * 4);
    w.active = cut.take(E * 4);
    w.n_active = cut.take(4);
    w.perm = cut.take(A * 4);
    w.inv_perm = cut.take(A * 4);
    w.plan_header = cut.take(PLAN_HEADER_INTS * 4);
    w.plan_seg = cut.take(sizeof(Segment) * (size_t)max_segments((int)E, (int)A));
    w.plan_pairs = cut.take(sizeof(PairEntry) * (size_t)max_segments((int)E, (int)A));
    w.plan_done = cut.take(4 * ((size_t)max_segments((int)E, (int)A) + max_shared_segments(T)));
    w.plan_done_shared_at = (size_t)max_segments((int)E, (int)A);
    w.x_sorted = cut.take(A * H * 2);
    w.h = cut.take(A * (size_t)c.inter * 2);
    w.h_shared = cut.take((size_t)T * c.shared_inter * 2);
    // y: [A,H], or while the down pass is short of work items partial planes of it
    const size_t A_split = ROUTED_SPLIT_MAX_PARTS * routed_split_max_rows(c, T);
    const size_t y_rows = A > A_split ? A : A_split;
    w.y = cut.take(y_rows * H * 2);
    w.y_shared = cut.take((size_t)T * H * 2 * shared_down_parts(c));
    w.rl_planes = cut.take(router_tc_plane_bytes(c, T));
    w.rl_partial = cut.take(router_tc_partial_bytes(c, T));
    w.small_logit_part = cut.take(layer_small_logit_part_bytes(c));
    w.small_h = cut.take(layer_small_h_bytes(c, T));
    w.total = cut.off;
    return w;
}

// ---------------------------------------------------------------------------------------
// Kernel launchers (each enqueues on `stream` and returns the launch error, if any).
// ---------------------------------------------------------------------------------------
// zero / zero_n: ints this kernel clears before any later kernel of the call may start (the
// shared expert's progress counters), or null; status: the workspace's status region, which
// the first kernel of a call initialises if it never was
cudaError_t launch_router_logits(const moe_config_t &c, const moe_weights_t &w,
                                 const __nv_bfloat16 *x, int T, float *logits,
                                 float *shared_scale, cudaStream_t s, int32_t *zero = nullptr,
                                 int zero_n = 0, int32_t *status = nullptr);
// The same on tcgen05 for large batches (router_logits_tc.cu): two launches (split of the fp32
// rows into bf16 planes, the contraction); planes / partial are the workspace regions of
// router_tc_plane_bytes / router_tc_partial_bytes.  The logits are left as partial sums
// [*chunks][T][E (+1 with the shared gate's row)] in `partial`: launch_route_topk_sum adds them.
cudaError_t launch_router_logits_tc(const moe_config_t &c, const moe_weights_t &w,
                                    const __nv_bfloat16 *x, int T, __nv_bfloat16 *planes,
                                    float *partial, cudaStream_t s, int32_t *zero, int zero_n,
                                    int32_t *status, int *launches, int *chunks);
cudaError_t launch_route_topk(const moe_config_t &c, const float *logits, int T, int32_t *idx,
                              float *wts, cudaStream_t s);
// the same from partial logits [chunks][T][R] (R = E, or E + 1 with the shared gate's row last):
// sums the chunks in chunk order, adds the bias, writes logits [T,E] (and shared_scale [T] if not
// null) and selects
cudaError_t launch_route_topk_sum(const moe_config_t &c, const float *partial, int chunks, int R,
                                  const float *bias, int T, float *logits, float *shared_scale,
                                  int32_t *idx, float *wts, cudaStream_t s);
cudaError_t launch_permute(const moe_config_t &c, const int32_t *idx, int T, int32_t *counts,
                           int32_t *offsets, int32_t *perm, int32_t *inv_perm, int32_t *active,
                           int32_t *n_active, cudaStream_t s, const PlanView *plan = nullptr,
                           int32_t *status = nullptr);
cudaError_t launch_plan(const moe_config_t &c, int T, const int32_t *offsets, int32_t *status,
                        PlanView plan, cudaStream_t s);
// expert FFN on the tensor cores, weights streamed by TMA (every group size):
// gate/up + SwiGLU -> h[row,:] (routed, sorted order) and h_shared[t,:];
// down projection  -> y[row,:] and y_shared[t,:]
cudaError_t launch_ffn_gateup(const moe_config_t &c, const moe_weights_t &w, const __nv_bfloat16 *x,
                              const __nv_bfloat16 *x_sorted, int T, PlanView plan, bool with_shared,
                              __nv_bfloat16 *h, __nv_bfloat16 *h_shared, int32_t *status,
                              cudaStream_t s);
cudaError_t launch_ffn_down(const moe_config_t &c, const moe_weights_t &w, int T, PlanView plan,
                            bool with_shared, const __nv_bfloat16 *h, const __nv_bfloat16 *h_shared,
                            __nv_bfloat16 *y, __nv_bfloat16 *y_shared, int shared_parts,
                            int routed_parts,
                            int32_t *status, cudaStream_t s);
// top-k, grouping, plan and gather of a small batch in one launch (replaces
// launch_route_topk + launch_permute + launch_gather_rows where it applies)
bool route_group_small_applies(const moe_config_t &c, int T);
cudaError_t launch_route_group_small(const moe_config_t &c, const float *logits,
                                     const __nv_bfloat16 *x, int T, int32_t *topk_idx, float *topk_w,
                                     int32_t *counts, int32_t *offsets, int32_t *perm,
                                     int32_t *inv_perm, int32_t *active, int32_t *n_active,
                                     int32_t *status, PlanView plan, __nv_bfloat16 *x_sorted,
                                     cudaStream_t s);
// one bounded wait on a word nothing sets (moe_selftest_wait_limit)
cudaError_t launch_wait_limit_selftest(int32_t *status, int32_t *never_set, int limit_us,
                                       cudaStream_t s);
// the same for the wait of the one-launch layer's counters; word [3] of the status region is set
// to 1 when that wait gave up
cudaError_t launch_tagged_wait_selftest(int32_t *status, int limit_us, cudaStream_t s);
// token rows in sorted order (the token operand of the routed gate/up tiles)
cudaError_t launch_gather_rows(const moe_config_t &c, const __nv_bfloat16 *x, const int32_t *perm,
                               int T, __nv_bfloat16 *x_sorted, cudaStream_t s);
// y and shared_y may hold `routed_parts` / `shared_parts` partial planes ([A,H] / [T,H]: k
// chunks of the down pass), summed here
cudaError_t launch_combine(const moe_config_t &c, const __nv_bfloat16 *y, int routed_parts,
                           const int32_t *inv_perm, const float *topk_w,
                           const __nv_bfloat16 *shared_y, int shared_parts,
                           const float *shared_scale, int T, __nv_bfloat16 *out, cudaStream_t s);

// Router logits, top-k, grouping, expert FFNs, shared expert and combine of at most four tokens
// in one cooperative launch; uses the regions status, logits .. inv_perm, small_logit_part and
// small_h of `L` in `ws`.
cudaError_t launch_layer_small(const moe_config_t &c, const moe_weights_t &w, const __nv_bfloat16 *x,
                               int T, __nv_bfloat16 *out, char *ws, const Workspace &L,
                               cudaStream_t s);

int sm_count();
bool pdl_enabled();  // programmatic dependent launch between the layer's kernels
// Test hook, read once per process from MOE_FF_RR: 0 / 1 forces the FFN kernels to deal the
// routed work as ranges / as single items, -1 (unset) leaves the choice to the host heuristic.
int schedule_override();
// The same for the ring geometry, from MOE_FF_WIDE: 0 / 1 forces segments of 128 / 256 rows.
int geometry_override();
// From MOE_SMALL_FUSED: 0 keeps calls of a few tokens on the chain of kernels every other call
// uses, -1 (unset) lets them take the one-launch kernel.
int small_layer_override();
// Token rows per segment of the routed groups for a call with T tokens: 128 or 256 (the plan and
// the FFN kernels of one call must agree on it).
int ffn_segment_rows(const moe_config_t &c, int T);

// Host-side argument checks and the FFN launch sequence shared by the entry points.
bool aligned16(const void *p);
moe_status_t check_config(const moe_config_t *c);
moe_status_t check_tokens(const moe_config_t *c, int64_t T);
moe_status_t check_device();
bool weights_ok(const moe_config_t *c, const moe_weights_t *w, bool need_router, bool need_experts);
PlanView plan_view(char *ws, const Workspace &L, int seg_rows);
moe_status_t read_and_clear_status(void *status_region);
// plan -> gate/up + SwiGLU -> down; uses the regions status, plan_*, h, h_shared of `L` in `ws`
moe_status_t run_ffn(const moe_config_t &c, const moe_weights_t &w, const __nv_bfloat16 *x, int T,
                     const int32_t *offsets, const int32_t *perm, __nv_bfloat16 *y,
                     __nv_bfloat16 *shared_y, char *ws, const Workspace &L, cudaStream_t s,
                     int &launches, bool plan_ready = false, int shared_parts = 1,
                     int routed_parts = 1, bool gathered = false);

// ---------------------------------------------------------------------------------------
// Device helpers.
// ---------------------------------------------------------------------------------------
#ifdef __CUDACC__

// An SM changes its L1 / shared-memory split only while it is idle.  The FFN kernels need the
// largest shared-memory split; if the small kernels before them ran with another one, an FFN
// CTA could not start on an SM as long as one of their CTAs is resident there (measured: the
// gate/up pass began only when the row gather had finished).  So every kernel of the library
// asks for the same, largest split (once per kernel).
void prefer_max_shared_carveout(const void *kernel);

// Launch with the programmatic-stream-serialization attribute: the kernel may begin while its
// predecessor in the stream is still running and must execute griddepcontrol.wait before it
// touches anything the predecessor produces.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t s, Args &&...args)
{
    prefer_max_shared_carveout(reinterpret_cast<const void *>(kernel));
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Programmatic dependent launch.  Every kernel of the layer is launched with launch_pdl and
// follows one discipline: it executes griddep_wait() before it reads or writes anything that
// a kernel of the same layer call produces or consumes, and before it exits; the first kernel
// of a call (router logits) and the gate/up pass trigger their dependents only after their
// own wait, so whatever a later kernel touches before ITS wait (the caller's inputs only) is
// older than the call itself.
// Blocks until the preceding kernel in the stream has completed and its writes are visible
// (returns at once when the kernel was not launched as a programmatic dependent).
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel in the stream start its own prologue.
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// 128-bit load of data that several warps of the CTA re-read (activations): cache in L1.
__device__ __forceinline__ uint4 ld_cached_v4(const void *p)
{
    uint4 v;
    asm volatile("ld.global.ca.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// One thread of the first kernel of a call, after its griddepcontrol.wait.
__device__ __forceinline__ void status_region_init(int32_t *status)
{
    if (status != nullptr && status[1] != STATUS_MAGIC) {
        status[0] = 0;
        status[1] = STATUS_MAGIC;
    }
}

// g * sigmoid(g) = g * (0.5 + 0.5 * tanh(g / 2)) with the hardware tanh: one special-function
// operation per value instead of two (exponential and reciprocal); its relative error, about
// 2^-11, is a quarter of the bf16 rounding the result goes through
__device__ __forceinline__ float silu_f(float g)
{
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * g));
    const float half_g = 0.5f * g;
    return fmaf(half_g, t, half_g);
}

#endif  // __CUDACC__

}  // namespace moe

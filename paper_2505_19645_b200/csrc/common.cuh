// Shared declarations of the CUDA path: workspace layout, segment plan, device helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "moe_verify.h"

namespace moe {

// ---------------------------------------------------------------------------------------
// Segment plan.  A segment is a run of at most SEG_TOKENS consecutive sorted rows that
// belong to one group (a routed expert, or the shared expert on rows of x itself).  The
// plan kernel derives the list from the grouping offsets on the device, so the host never
// needs the data-dependent counts and no launch waits for a copy.
// ---------------------------------------------------------------------------------------
constexpr int SEG_TOKENS = 32;      // rows per segment of the streaming path (4 MMA n-chunks)
constexpr int TC_SEG_TOKENS = 128;  // rows per segment of the tensor-core path (UMMA N)
constexpr int TC_MIN_ROWS = 32;     // groups with more rows than this take the tensor-core path
constexpr int PLAN_HEADER_INTS = 16;

struct Segment {
    int32_t expert;  // routed expert id, or -1 for the shared expert
    int32_t row0;    // first sorted row (routed) or first token row (shared)
    int32_t n;       // rows in this segment, 1..SEG_TOKENS
    int32_t pad;
};

// plan header (ints): [0] routed / [1] shared streaming segments,
//                     [2] routed / [3] shared tensor-core segments
struct PlanView {
    int32_t *header;
    Segment *routed;     // capacity max_routed_segments()
    Segment *shared;     // capacity max_shared_segments()
    Segment *tc_routed;  // capacity max_tc_routed_segments()
    Segment *tc_shared;  // capacity max_tc_shared_segments()
};

__host__ __device__ inline int max_routed_segments(int E, int A)
{
    return E + A / SEG_TOKENS + 1;
}
__host__ __device__ inline int max_shared_segments(int T)
{
    return (T + SEG_TOKENS - 1) / SEG_TOKENS;
}
__host__ __device__ inline int max_tc_routed_segments(int E, int A)
{
    return E + A / TC_SEG_TOKENS + 1;
}
__host__ __device__ inline int max_tc_shared_segments(int T)
{
    return (T + TC_SEG_TOKENS - 1) / TC_SEG_TOKENS;
}

// ---------------------------------------------------------------------------------------
// Workspace layout (every region 256-byte aligned).
// ---------------------------------------------------------------------------------------
struct Workspace {
    size_t status;        // int32[64]: [0] device status word
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
    size_t plan_routed;   // Segment[max_routed_segments]
    size_t plan_shared;   // Segment[max_shared_segments]
    size_t plan_tc_routed;  // Segment[max_tc_routed_segments]
    size_t plan_tc_shared;  // Segment[max_tc_shared_segments]
    size_t x_sorted;      // bf16 [A, H]      token rows in sorted order (tensor-core path)
    size_t h;             // bf16 [A, I]      SwiGLU intermediate, sorted order
    size_t h_shared;      // bf16 [T, I_s]
    size_t y;             // bf16 [A, H]      expert outputs, sorted order
    size_t y_shared;      // bf16 [T, H]
    size_t total;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline Workspace workspace_layout(const moe_config_t &c, int T)
{
    Workspace w{};
    const size_t A = (size_t)T * c.top_k, E = c.n_experts, H = c.hidden;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    w.status = take(64 * 4);
    w.logits = take((size_t)T * E * 4);
    w.topk_idx = take(A * 4);
    w.topk_w = take(A * 4);
    w.shared_scale = take((size_t)T * 4);
    w.counts = take(E * 4);
    w.offsets = take((E + 1) * 4);
    w.active = take(E * 4);
    w.n_active = take(4);
    w.perm = take(A * 4);
    w.inv_perm = take(A * 4);
    w.plan_header = take(PLAN_HEADER_INTS * 4);
    w.plan_routed = take(sizeof(Segment) * (size_t)max_routed_segments((int)E, (int)A));
    w.plan_shared = take(sizeof(Segment) * (size_t)max_shared_segments(T));
    w.plan_tc_routed = take(sizeof(Segment) * (size_t)max_tc_routed_segments((int)E, (int)A));
    w.plan_tc_shared = take(sizeof(Segment) * (size_t)max_tc_shared_segments(T));
    w.x_sorted = take(T > TC_MIN_ROWS ? A * H * 2 : 0);
    w.h = take(A * (size_t)c.inter * 2);
    w.h_shared = take((size_t)T * c.shared_inter * 2);
    w.y = take(A * H * 2);
    w.y_shared = take((size_t)T * H * 2);
    w.total = off;
    return w;
}

// ---------------------------------------------------------------------------------------
// Kernel launchers (each enqueues on `stream` and returns the launch error, if any).
// ---------------------------------------------------------------------------------------
struct LaunchCounter {
    int n = 0;
};

cudaError_t launch_router_logits(const moe_config_t &c, const moe_weights_t &w,
                                 const __nv_bfloat16 *x, int T, float *logits,
                                 float *shared_scale, cudaStream_t s);
cudaError_t launch_route_topk(const moe_config_t &c, const float *logits, int T, int32_t *idx,
                              float *wts, cudaStream_t s);
cudaError_t launch_permute(const moe_config_t &c, const int32_t *idx, int T, int32_t *counts,
                           int32_t *offsets, int32_t *perm, int32_t *inv_perm, int32_t *active,
                           int32_t *n_active, cudaStream_t s, const PlanView *plan = nullptr,
                           bool with_shared = false, int tc_min_rows = TC_MIN_ROWS,
                           int32_t *status = nullptr);
cudaError_t launch_plan(const moe_config_t &c, int T, const int32_t *offsets, bool with_shared,
                        int tc_min_rows, int32_t *status, PlanView plan, cudaStream_t s);
// tensor-core path (groups with more than TC_MIN_ROWS rows)
cudaError_t launch_gather_rows(const moe_config_t &c, const __nv_bfloat16 *x, const int32_t *perm,
                               int T, __nv_bfloat16 *x_sorted, cudaStream_t s);
cudaError_t launch_ffn_tc_gateup(const moe_config_t &c, const moe_weights_t &w,
                                 const __nv_bfloat16 *x, const __nv_bfloat16 *x_sorted, int T,
                                 PlanView plan, bool with_shared, __nv_bfloat16 *h,
                                 __nv_bfloat16 *h_shared, int32_t *status, cudaStream_t s);
cudaError_t launch_ffn_tc_down(const moe_config_t &c, const moe_weights_t &w, int T, PlanView plan,
                               bool with_shared, const __nv_bfloat16 *h,
                               const __nv_bfloat16 *h_shared, __nv_bfloat16 *y,
                               __nv_bfloat16 *y_shared, int32_t *status, cudaStream_t s);
// gate/up + SwiGLU for every segment of the plan: h[row,:] (routed) and h_shared[row,:]
cudaError_t launch_ffn_stream_gateup(const moe_config_t &c, const moe_weights_t &w,
                                     const __nv_bfloat16 *x, int T, const int32_t *perm,
                                     PlanView plan, bool with_shared, __nv_bfloat16 *h,
                                     __nv_bfloat16 *h_shared, cudaStream_t s);
// down projection for every segment: y[row,:] and y_shared[row,:]
cudaError_t launch_ffn_stream_down(const moe_config_t &c, const moe_weights_t &w, int T,
                                   PlanView plan, bool with_shared, const __nv_bfloat16 *h,
                                   const __nv_bfloat16 *h_shared, __nv_bfloat16 *y,
                                   __nv_bfloat16 *y_shared, cudaStream_t s);
cudaError_t launch_combine(const moe_config_t &c, const __nv_bfloat16 *y, const int32_t *inv_perm,
                           const float *topk_w, const __nv_bfloat16 *shared_y,
                           const float *shared_scale, int T, __nv_bfloat16 *out, cudaStream_t s);

int sm_count();

// Host-side argument checks and the FFN launch sequence shared by the entry points.
bool aligned16(const void *p);
moe_status_t check_config(const moe_config_t *c);
moe_status_t check_tokens(const moe_config_t *c, int64_t T);
moe_status_t check_device();
bool weights_ok(const moe_config_t *c, const moe_weights_t *w, bool need_router, bool need_experts);
PlanView plan_view(char *ws, const Workspace &L);
// plan -> gate/up + SwiGLU -> down; uses the regions status, plan_*, h, h_shared of `L` in `ws`
moe_status_t run_ffn(const moe_config_t &c, const moe_weights_t &w, const __nv_bfloat16 *x, int T,
                     const int32_t *offsets, const int32_t *perm, __nv_bfloat16 *y,
                     __nv_bfloat16 *shared_y, char *ws, const Workspace &L, cudaStream_t s,
                     int &launches, bool plan_ready = false);

// ---------------------------------------------------------------------------------------
// Device helpers.
// ---------------------------------------------------------------------------------------
#ifdef __CUDACC__

// 128-bit streaming load: weights are read exactly once, keep them out of L1.
__device__ __forceinline__ uint4 ld_stream_v4(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

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

__device__ __forceinline__ float silu_f(float g) { return g / (1.0f + __expf(-g)); }

#endif  // __CUDACC__

}  // namespace moe

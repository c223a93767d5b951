// Token-to-expert grouping: histogram, exclusive scan, stable placement, active-expert list,
// and the segment plan the FFN kernels iterate over.
#include "common.cuh"

namespace moe {

constexpr int PERM_THREADS = 1024;  // 32 warps: one warp places one expert

// Exclusive scan of vals[0..n) (n <= MOE_MAX_EXPERTS <= blockDim.x) in shared memory;
// returns the total in *total.  All threads of the block must call it.
__device__ void block_exclusive_scan(int *vals, int *tmp, int n, int *total)
{
    const int tid = threadIdx.x;
    int v = tid < n ? vals[tid] : 0;
    if (tid < MOE_MAX_EXPERTS)
        tmp[tid] = v;
    __syncthreads();
    for (int off = 1; off < MOE_MAX_EXPERTS; off <<= 1) {
        int add = 0;
        if (tid < MOE_MAX_EXPERTS && tid >= off)
            add = tmp[tid - off];
        __syncthreads();
        if (tid < MOE_MAX_EXPERTS)
            tmp[tid] += add;
        __syncthreads();
    }
    if (tid < n)
        vals[tid] = tmp[tid] - v;  // inclusive -> exclusive
    if (tid == 0)
        *total = tmp[MOE_MAX_EXPERTS - 1];
    __syncthreads();
}

// Every CTA rebuilds the (tiny) histogram and scan for itself, so no grid-wide
// dependency is needed; CTA b then places experts 32b .. 32b+31, one warp each, walking
// the assignments in ascending order (ballot + prefix popcount) -- stable by construction,
// no atomics decide a position.  CTA 0 also writes counts / offsets / active / n_active.
__global__ void __launch_bounds__(PERM_THREADS)
permute_kernel(const int32_t *__restrict__ topk_idx, int A, int E, int32_t *__restrict__ counts,
               int32_t *__restrict__ offsets, int32_t *__restrict__ perm,
               int32_t *__restrict__ inv_perm, int32_t *__restrict__ active,
               int32_t *__restrict__ n_active, int T, int with_shared,
               int32_t *__restrict__ status, int32_t *__restrict__ plan_header,
               Segment *__restrict__ plan_routed, Segment *__restrict__ plan_shared)
{
    __shared__ int hist[MOE_MAX_EXPERTS];
    __shared__ int offs[MOE_MAX_EXPERTS];
    __shared__ int flag[MOE_MAX_EXPERTS];
    __shared__ int tmp[MOE_MAX_EXPERTS];
    __shared__ int total;
    const int tid = threadIdx.x;
    if (tid < MOE_MAX_EXPERTS)
        hist[tid] = 0;
    __syncthreads();
    for (int a = tid; a < A; a += PERM_THREADS) {
        const int e = topk_idx[a];
        if (e >= 0 && e < E)
            atomicAdd(&hist[e], 1);  // a count does not depend on the order of the adds
    }
    __syncthreads();
    if (tid < MOE_MAX_EXPERTS)
        offs[tid] = tid < E ? hist[tid] : 0;
    __syncthreads();
    block_exclusive_scan(offs, tmp, E, &total);

    if (blockIdx.x == 0) {
        if (tid < E) {
            counts[tid] = hist[tid];
            offsets[tid] = offs[tid];
        }
        if (tid == 0)
            offsets[E] = total;
        if (tid < MOE_MAX_EXPERTS)
            flag[tid] = (tid < E && hist[tid] > 0) ? 1 : 0;
        __syncthreads();
        int my_flag = tid < E ? flag[tid] : 0;
        block_exclusive_scan(flag, tmp, E, &total);
        if (tid < E && my_flag)
            active[flag[tid]] = tid;
        if (tid < E && tid >= total)
            active[tid] = -1;
        if (tid == 0)
            n_active[0] = total;
        // Inside moe_verify_layer the segment plan of the FFN kernels is written here as
        // well (same content as plan_kernel), which saves a launch.
        if (plan_header != nullptr) {
            __syncthreads();
            const int cnt = tid < E ? hist[tid] : 0;
            if (tid < MOE_MAX_EXPERTS)
                flag[tid] = (cnt + SEG_TOKENS - 1) / SEG_TOKENS;
            __syncthreads();
            block_exclusive_scan(flag, tmp, E, &total);
            if (tid < E) {
                int at = flag[tid];
                const int row0 = offs[tid];
                for (int r = 0; r < cnt; r += SEG_TOKENS) {
                    Segment sg;
                    sg.expert = tid;
                    sg.row0 = row0 + r;
                    sg.n = min(SEG_TOKENS, cnt - r);
                    sg.pad = 0;
                    plan_routed[at++] = sg;
                }
            }
            const int n_shared = with_shared ? (T + SEG_TOKENS - 1) / SEG_TOKENS : 0;
            for (int i = tid; i < n_shared; i += PERM_THREADS) {
                Segment sg;
                sg.expert = -1;
                sg.row0 = i * SEG_TOKENS;
                sg.n = min(SEG_TOKENS, T - i * SEG_TOKENS);
                sg.pad = 0;
                plan_shared[i] = sg;
            }
            if (tid == 0) {
                plan_header[0] = total;
                plan_header[1] = n_shared;
                status[0] = 0;
            }
        }
    }

    const int warp = tid >> 5, lane = tid & 31;
    const int e = blockIdx.x * 32 + warp;
    if (e >= E || hist[e] == 0)
        return;
    int base = offs[e];
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int a0 = 0; a0 < A; a0 += 128) {
        int ev[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int a = a0 + u * 32 + lane;
            ev[u] = a < A ? topk_idx[a] : -1;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int a = a0 + u * 32 + lane;
            const bool hit = ev[u] == e;
            const uint32_t m = __ballot_sync(0xffffffffu, hit);
            if (hit) {
                const int pos = base + __popc(m & lt_mask);
                perm[pos] = a;
                inv_perm[a] = pos;
            }
            base += __popc(m);
        }
    }
}

cudaError_t launch_permute(const moe_config_t &c, const int32_t *idx, int T, int32_t *counts,
                           int32_t *offsets, int32_t *perm, int32_t *inv_perm, int32_t *active,
                           int32_t *n_active, cudaStream_t s, const PlanView *plan,
                           bool with_shared, int32_t *status)
{
    const int E = c.n_experts;
    const int blocks = (E + 31) / 32;
    permute_kernel<<<blocks, PERM_THREADS, 0, s>>>(
        idx, T * c.top_k, E, counts, offsets, perm, inv_perm, active, n_active, T,
        with_shared ? 1 : 0, status, plan ? plan->header : nullptr, plan ? plan->routed : nullptr,
        plan ? plan->shared : nullptr);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Segment plan: cut every expert's run of sorted rows into segments of <= SEG_TOKENS rows.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(MOE_MAX_EXPERTS)
plan_kernel(const int32_t *__restrict__ offsets, int E, int T, int with_shared,
            int32_t *__restrict__ status, int32_t *__restrict__ header,
            Segment *__restrict__ routed, Segment *__restrict__ shared)
{
    __shared__ int nseg[MOE_MAX_EXPERTS];
    __shared__ int tmp[MOE_MAX_EXPERTS];
    __shared__ int total;
    const int tid = threadIdx.x;
    int row0 = 0, cnt = 0;
    if (tid < E) {
        row0 = offsets[tid];
        cnt = offsets[tid + 1] - row0;
    }
    nseg[tid] = (cnt + SEG_TOKENS - 1) / SEG_TOKENS;
    __syncthreads();
    block_exclusive_scan(nseg, tmp, E, &total);
    if (tid < E) {
        int at = nseg[tid];
        for (int r = 0; r < cnt; r += SEG_TOKENS) {
            Segment sg;
            sg.expert = tid;
            sg.row0 = row0 + r;
            sg.n = min(SEG_TOKENS, cnt - r);
            sg.pad = 0;
            routed[at++] = sg;
        }
    }
    const int n_shared = with_shared ? (T + SEG_TOKENS - 1) / SEG_TOKENS : 0;
    for (int i = tid; i < n_shared; i += blockDim.x) {
        Segment sg;
        sg.expert = -1;
        sg.row0 = i * SEG_TOKENS;
        sg.n = min(SEG_TOKENS, T - i * SEG_TOKENS);
        sg.pad = 0;
        shared[i] = sg;
    }
    if (tid == 0) {
        header[0] = total;
        header[1] = n_shared;
        status[0] = 0;  // device status word: cleared at the start of every FFN pass
    }
}

cudaError_t launch_plan(const moe_config_t &c, int T, const int32_t *offsets, bool with_shared,
                        int32_t *status, PlanView plan, cudaStream_t s)
{
    plan_kernel<<<1, MOE_MAX_EXPERTS, 0, s>>>(offsets, c.n_experts, T, with_shared ? 1 : 0, status,
                                              plan.header, plan.routed, plan.shared);
    return cudaGetLastError();
}

}  // namespace moe

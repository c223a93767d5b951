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

// Segment plan from per-expert counts and offsets held in shared memory.  A group (expert, or
// the shared expert with its T rows) with at most tc_min_rows rows is cut into streaming
// segments of <= SEG_TOKENS rows; a larger group into tensor-core segments of <= TC_SEG_TOKENS
// rows.  All threads of the block must call it; scan/tmp/total are shared scratch.
__device__ void build_plan(const int *cnt_sh, const int *off_sh, int *scan, int *tmp, int *total,
                           int E, int T, int with_shared, int tc_min_rows, int32_t *status,
                           PlanView plan)
{
    const int tid = threadIdx.x;
    const int cnt = tid < E ? cnt_sh[tid] : 0;
    const int row0 = tid < E ? off_sh[tid] : 0;
    const bool tc = cnt > tc_min_rows;
    for (int pass = 0; pass < 2; ++pass) {
        const int seg_rows = pass == 0 ? SEG_TOKENS : TC_SEG_TOKENS;
        const bool mine = cnt > 0 && (pass == 0 ? !tc : tc);
        __syncthreads();
        if (tid < MOE_MAX_EXPERTS)
            scan[tid] = mine ? (cnt + seg_rows - 1) / seg_rows : 0;
        __syncthreads();
        block_exclusive_scan(scan, tmp, E, total);
        Segment *list = pass == 0 ? plan.routed : plan.tc_routed;
        if (mine) {
            int at = scan[tid];
            for (int r = 0; r < cnt; r += seg_rows) {
                Segment sg;
                sg.expert = tid;
                sg.row0 = row0 + r;
                sg.n = min(seg_rows, cnt - r);
                sg.pad = 0;
                list[at++] = sg;
            }
        }
        if (tid == 0)
            plan.header[pass == 0 ? 0 : 2] = *total;
    }
    const bool shared_tc = T > tc_min_rows;
    const int seg_rows = shared_tc ? TC_SEG_TOKENS : SEG_TOKENS;
    const int n_shared = with_shared ? (T + seg_rows - 1) / seg_rows : 0;
    Segment *slist = shared_tc ? plan.tc_shared : plan.shared;
    for (int i = tid; i < n_shared; i += blockDim.x) {
        Segment sg;
        sg.expert = -1;
        sg.row0 = i * seg_rows;
        sg.n = min(seg_rows, T - i * seg_rows);
        sg.pad = 0;
        slist[i] = sg;
    }
    if (tid == 0) {
        plan.header[1] = shared_tc ? 0 : n_shared;
        plan.header[3] = shared_tc ? n_shared : 0;
        status[0] = 0;  // device status word: cleared at the start of every FFN pass
    }
}

// Every CTA rebuilds the (tiny) histogram and scan for itself, so no grid-wide
// dependency is needed; CTA b then places experts 32b .. 32b+31, one warp each, walking
// the assignments in ascending order (ballot + prefix popcount) -- stable by construction,
// no atomics decide a position.  CTA 0 also writes counts / offsets / active / n_active and,
// inside moe_verify_layer, the FFN segment plan (one launch fewer).
__global__ void __launch_bounds__(PERM_THREADS)
permute_kernel(const int32_t *__restrict__ topk_idx, int A, int E, int32_t *__restrict__ counts,
               int32_t *__restrict__ offsets, int32_t *__restrict__ perm,
               int32_t *__restrict__ inv_perm, int32_t *__restrict__ active,
               int32_t *__restrict__ n_active, int T, int with_shared, int tc_min_rows,
               int32_t *__restrict__ status, PlanView plan)
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
        if (plan.header != nullptr)
            build_plan(hist, offs, flag, tmp, &total, E, T, with_shared, tc_min_rows, status, plan);
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
                           bool with_shared, int tc_min_rows, int32_t *status)
{
    const int E = c.n_experts;
    const int blocks = (E + 31) / 32;
    PlanView pv{};
    if (plan)
        pv = *plan;
    permute_kernel<<<blocks, PERM_THREADS, 0, s>>>(idx, T * c.top_k, E, counts, offsets, perm,
                                                   inv_perm, active, n_active, T,
                                                   with_shared ? 1 : 0, tc_min_rows, status, pv);
    return cudaGetLastError();
}

// Stand-alone plan (moe_grouped_swiglu gets its offsets from the caller).
__global__ void __launch_bounds__(MOE_MAX_EXPERTS)
plan_kernel(const int32_t *__restrict__ offsets, int E, int T, int with_shared, int tc_min_rows,
            int32_t *__restrict__ status, PlanView plan)
{
    __shared__ int cnt[MOE_MAX_EXPERTS];
    __shared__ int offs[MOE_MAX_EXPERTS];
    __shared__ int scan[MOE_MAX_EXPERTS];
    __shared__ int tmp[MOE_MAX_EXPERTS];
    __shared__ int total;
    const int tid = threadIdx.x;
    int row0 = 0, n = 0;
    if (tid < E) {
        row0 = offsets[tid];
        n = offsets[tid + 1] - row0;
    }
    cnt[tid] = n;
    offs[tid] = row0;
    __syncthreads();
    build_plan(cnt, offs, scan, tmp, &total, E, T, with_shared, tc_min_rows, status, plan);
}

cudaError_t launch_plan(const moe_config_t &c, int T, const int32_t *offsets, bool with_shared,
                        int tc_min_rows, int32_t *status, PlanView plan, cudaStream_t s)
{
    plan_kernel<<<1, MOE_MAX_EXPERTS, 0, s>>>(offsets, c.n_experts, T, with_shared ? 1 : 0,
                                              tc_min_rows, status, plan);
    return cudaGetLastError();
}

}  // namespace moe

// Token-to-expert grouping: histogram, exclusive scan, stable placement, active-expert list,
// and the segment plan the FFN kernels iterate over.
#include "route_topk.cuh"

namespace moe {

constexpr int PERM_THREADS = 1024;  // assignments per CTA, one per thread
constexpr int ROUTE_SMALL_TOKENS = 32;   // one warp per token in a CTA of PERM_THREADS
constexpr int ROUTE_SMALL_ASSIGN = 512;  // = ROUTE_SMALL_TOKENS * MOE_MAX_TOPK

// Exclusive scan of vals[0..n) (n <= MOE_MAX_EXPERTS <= blockDim.x) in shared memory;
// returns the total in *total.  All threads of the block must call it.  Warp shuffles inside
// each group of 32 entries, then one warp scans the 16 group sums (tmp).
__device__ void block_exclusive_scan(int *vals, int *tmp, int n, int *total)
{
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    constexpr int NW = MOE_MAX_EXPERTS / 32;
    int v = 0, incl = 0;
    if (wid < NW) {
        v = tid < n ? vals[tid] : 0;
        incl = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off)
                incl += o;
        }
        if (lane == 31)
            tmp[wid] = incl;
    }
    __syncthreads();
    if (wid == 0) {
        const int w = lane < NW ? tmp[lane] : 0;
        int wi = w;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, wi, off);
            if (lane >= off)
                wi += o;
        }
        if (lane < NW)
            tmp[lane] = wi - w;  // exclusive offset of each group
        if (lane == NW - 1)
            *total = wi;
    }
    __syncthreads();
    if (wid < NW && tid < n)
        vals[tid] = tmp[wid] + incl - v;
    __syncthreads();
}

// Segment plan from per-expert counts and offsets held in shared memory: one entry per
// segment of plan.seg_rows rows of every activated expert, in ascending expert order.  All
// threads of the block must call it; scan/tmp/total are shared scratch.
__device__ void build_plan(const int *cnt_sh, const int *off_sh, int *scan, int *tmp, int *total,
                           int E, int32_t *status, PlanView plan)
{
    const int tid = threadIdx.x;
    const int cnt = tid < E ? cnt_sh[tid] : 0;
    const int row0 = tid < E ? off_sh[tid] : 0;
    const int nseg = (cnt + plan.seg_rows - 1) / plan.seg_rows;
    __syncthreads();
    if (tid < MOE_MAX_EXPERTS)
        scan[tid] = nseg;
    __syncthreads();
    block_exclusive_scan(scan, tmp, E, total);
    if (nseg > 0) {
        const int first = scan[tid];
        Segment sg;
        sg.expert = tid;
        sg.row0 = row0;
        sg.n = cnt;
        sg.first_seg = first;
        for (int i = 0; i < nseg; ++i) {
            plan.seg[first + i] = sg;
            plan.done_routed[first + i] = 0;
        }
    }
    if (tid == 0)
        plan.header[0] = *total;
    // the item list: one entry per segment, carrying its group
    const int first = nseg > 0 ? scan[tid] : 0;
    for (int q = 0; q < nseg; ++q) {
        PairEntry pe;
        pe.expert = tid;
        pe.row0 = row0;
        pe.n = cnt;
        pe.first_seg = first;
        pe.seg = first + q;
        pe.pad[0] = pe.pad[1] = pe.pad[2] = 0;
        plan.pairs[first + q] = pe;
    }
    if (tid == 0) {
        plan.header[1] = *total;
        plan.header[2] = 0;  // work claimed so far by the gate/up pass ...
        plan.header[3] = 0;  // ... and by the down pass
    }
}

// counts / offsets / active / n_active from the histogram and its exclusive scan (shared
// memory, `total` = number of assignments) and, if asked for, the FFN segment plan.  All
// threads of the block must call it; flag/tmp are shared scratch of MOE_MAX_EXPERTS ints.
__device__ void write_tables(int *hist, int *offs, int *flag, int *tmp, int *total, int E,
                             int32_t *counts, int32_t *offsets, int32_t *active, int32_t *n_active,
                             int32_t *status, PlanView plan)
{
    const int tid = threadIdx.x;
    __syncthreads();
    if (tid < E) {
        counts[tid] = hist[tid];
        offsets[tid] = offs[tid];
    }
    if (tid == 0)
        offsets[E] = *total;
    if (tid < MOE_MAX_EXPERTS)
        flag[tid] = (tid < E && hist[tid] > 0) ? 1 : 0;
    __syncthreads();
    const int my_flag = tid < E ? flag[tid] : 0;
    block_exclusive_scan(flag, tmp, E, total);
    if (tid < E && my_flag)
        active[flag[tid]] = tid;
    if (tid < E && tid >= *total)
        active[tid] = -1;
    if (tid == 0)
        n_active[0] = *total;
    if (plan.header != nullptr)
        build_plan(hist, offs, flag, tmp, total, E, status, plan);
}

// Adds one to hist[e] for every lane with a valid e.  With few experts a plain per-lane
// atomic would serialise the block on a handful of counters, so the lanes of a warp that hold
// the same expert are combined first (one atomic per distinct expert); with many experts the
// match itself (one round per distinct value) costs more than the rare conflict.
// All lanes of the warp must call it; `few` is uniform.
__device__ __forceinline__ void warp_histogram_add(int *hist, int e, bool valid, bool few)
{
    if (few) {
        const uint32_t peers = __match_any_sync(0xffffffffu, valid ? e : -1);
        if (valid && (threadIdx.x & 31) == __ffs(peers) - 1)
            atomicAdd(&hist[e], __popc(peers));
    } else if (valid) {
        atomicAdd(&hist[e], 1);  // a count does not depend on the order of the adds
    }
}

// Stable counting sort of the assignments by expert.  CTA b owns assignments
// [b * 1024, b * 1024 + 1024), one per thread.  Every CTA rebuilds the (small) histograms it
// needs for itself -- all assignments for the expert offsets, those before its own chunk for
// its starting ranks -- so no grid-wide dependency is needed.  Inside the chunk an
// assignment's rank among those of its expert is (earlier warps' counts, from a per-warp
// table) + (earlier lanes of its warp, from a match mask): ascending assignment id within
// every expert by construction, no atomics decide a position.  One more CTA, which owns no
// chunk, writes counts / offsets / active / n_active and, inside moe_verify_layer, the FFN
// segment plan at the same time.
__global__ void __launch_bounds__(PERM_THREADS)
permute_kernel(const int32_t *__restrict__ topk_idx, int A, int E, int32_t *__restrict__ counts,
               int32_t *__restrict__ offsets, int32_t *__restrict__ perm,
               int32_t *__restrict__ inv_perm, int32_t *__restrict__ active,
               int32_t *__restrict__ n_active, int32_t *__restrict__ status, PlanView plan)
{
    __shared__ int hist[MOE_MAX_EXPERTS];    // all assignments
    __shared__ int before[MOE_MAX_EXPERTS];  // assignments of earlier chunks
    __shared__ int offs[MOE_MAX_EXPERTS];
    __shared__ int tmp[MOE_MAX_EXPERTS];
    __shared__ uint16_t wcount[PERM_THREADS / 32][MOE_MAX_EXPERTS];  // per warp of this chunk
    __shared__ int total;
    griddep_launch();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // the last CTA owns no chunk: it writes the tables and the plan while the others place
    const bool tables_cta = blockIdx.x == gridDim.x - 1;
    const int chunk0 = tables_cta ? 0 : blockIdx.x * PERM_THREADS;
    if (tid < MOE_MAX_EXPERTS) {
        hist[tid] = 0;
        before[tid] = 0;
    }
    for (int i = tid; i < (PERM_THREADS / 32) * MOE_MAX_EXPERTS / 2; i += PERM_THREADS)
        reinterpret_cast<uint32_t *>(&wcount[0][0])[i] = 0u;
    griddep_wait();  // the expert indices come from the preceding kernel
    __syncthreads();
    const bool few = E <= 32;
    for (int a0 = 0; a0 < A; a0 += PERM_THREADS) {
        const int a = a0 + tid;
        const int e = a < A ? topk_idx[a] : -1;
        const bool valid = e >= 0 && e < E;
        warp_histogram_add(hist, e, valid, few);
        if (a0 < chunk0)
            warp_histogram_add(before, e, valid, few);
    }
    // this thread's assignment: rank inside its warp, and its warp's counts
    const int my_a = chunk0 + tid;
    const int my_e = !tables_cta && my_a < A ? topk_idx[my_a] : -1;
    const bool my_valid = my_e >= 0 && my_e < E;
    const uint32_t peers = __match_any_sync(0xffffffffu, my_valid ? my_e : -1);
    const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
    if (my_valid && lane == __ffs(peers) - 1)
        wcount[warp][my_e] = (uint16_t)__popc(peers);
    __syncthreads();
    if (tid < MOE_MAX_EXPERTS)
        offs[tid] = tid < E ? hist[tid] : 0;
    __syncthreads();
    block_exclusive_scan(offs, tmp, E, &total);

    if (my_valid) {
        int pos = offs[my_e] + before[my_e] + rank_in_warp;
        for (int w = 0; w < warp; ++w)
            pos += wcount[w][my_e];
        perm[pos] = my_a;
        inv_perm[my_a] = pos;
    }

    if (tables_cta)  // this CTA counted no earlier chunk: `before` is free (all zero)
        write_tables(hist, offs, before, tmp, &total, E, counts, offsets, active, n_active, status, plan);
}

cudaError_t launch_permute(const moe_config_t &c, const int32_t *idx, int T, int32_t *counts,
                           int32_t *offsets, int32_t *perm, int32_t *inv_perm, int32_t *active,
                           int32_t *n_active, cudaStream_t s, const PlanView *plan, int32_t *status)
{
    const int A = T * c.top_k;
    const int blocks = (A + PERM_THREADS - 1) / PERM_THREADS + 1;  // + the tables CTA
    PlanView pv{};
    if (plan)
        pv = *plan;
    return launch_pdl(permute_kernel, dim3(blocks), dim3(PERM_THREADS), 0, s, idx, A, c.n_experts,
                      counts, offsets, perm, inv_perm, active, n_active, status, pv);
}

// Routing of a small batch in one launch: top-k, grouping, segment plan and the gather of
// the token rows into sorted order, for T <= ROUTE_SMALL_TOKENS tokens and at most
// ROUTE_SMALL_ASSIGN assignments.  Every CTA repeats the (tiny) top-k and counting sort for
// itself, so no CTA waits for another: CTA 0 writes topk_idx / topk_w / perm / inv_perm, CTA 1
// the tables and the plan, and the others copy the rows x[perm[r] / k] -> x_sorted[r], row r
// on CTA 2 + r mod (gridDim.x - 2).  Results are those of route_topk_kernel, permute_kernel
// and gather_rows_kernel run one after the other, with two launch boundaries fewer on the
// path from the logits to the first routed tile.
template <int VPL>
__global__ void __launch_bounds__(PERM_THREADS)
route_group_small_kernel(const float *__restrict__ logits, const __nv_bfloat16 *__restrict__ x,
                         int T, int H, int E, int k, int score_fn, int renormalize,
                         float routed_scale, int32_t *__restrict__ topk_idx,
                         float *__restrict__ topk_w, int32_t *__restrict__ counts,
                         int32_t *__restrict__ offsets, int32_t *__restrict__ perm,
                         int32_t *__restrict__ inv_perm, int32_t *__restrict__ active,
                         int32_t *__restrict__ n_active, int32_t *__restrict__ status,
                         PlanView plan, __nv_bfloat16 *__restrict__ x_sorted)
{
    __shared__ int hist[MOE_MAX_EXPERTS];
    __shared__ int offs[MOE_MAX_EXPERTS];
    __shared__ int tmp[MOE_MAX_EXPERTS];
    __shared__ int flag[MOE_MAX_EXPERTS];
    __shared__ uint16_t wcount[ROUTE_SMALL_ASSIGN / 32][MOE_MAX_EXPERTS];
    __shared__ int expert_of[ROUTE_SMALL_ASSIGN];  // by assignment t * k + j
    __shared__ int token_of[ROUTE_SMALL_ASSIGN];   // by sorted row
    __shared__ int total;
    griddep_launch();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int A = T * k;
    if (tid < MOE_MAX_EXPERTS)
        hist[tid] = 0;
    for (int i = tid; i < (ROUTE_SMALL_ASSIGN / 32) * MOE_MAX_EXPERTS / 2; i += PERM_THREADS)
        reinterpret_cast<uint32_t *>(&wcount[0][0])[i] = 0u;
    griddep_wait();  // the logits come from the preceding kernel

    // top-k: warp w selects for token w
    if (warp < T) {
        int sel_i;
        float sel_w;
        warp_route_topk<VPL>(logits + (size_t)warp * E, E, k, score_fn, renormalize, routed_scale,
                             lane, sel_i, sel_w);
        if (lane < k) {
            expert_of[warp * k + lane] = sel_i;
            if (blockIdx.x == 0) {
                topk_idx[warp * k + lane] = sel_i;
                topk_w[warp * k + lane] = sel_w;
            }
        }
    }
    __syncthreads();

    if (A <= 32) {
        // At most a warp's worth of assignments: one warp sorts them with shuffles and every
        // thread derives its expert's table entries from the (few) assignments directly --
        // two barriers in all instead of the scans below.
        if (warp == 0) {
            const int e = lane < A ? expert_of[lane] : -1;
            const uint32_t peers = __match_any_sync(0xffffffffu, e);
            const int rank = __popc(peers & ((1u << lane) - 1u));
            int less = 0;
#pragma unroll
            for (int src = 0; src < 32; ++src) {
                const int other = __shfl_sync(0xffffffffu, e, src);
                less += (other >= 0 && other < e) ? 1 : 0;
            }
            flag[lane] = (e >= 0 && lane == __ffs(peers) - 1) ? 1 : 0;  // first of its expert
            if (e >= 0) {
                const int pos = less + rank;  // stable: ascending assignment id inside an expert
                token_of[pos] = lane / k;
                if (blockIdx.x == 0) {
                    perm[pos] = lane;
                    inv_perm[lane] = pos;
                }
            }
        }
        __syncthreads();
        if (blockIdx.x == 1) {
            int cnt = 0, off = 0, arank = 0, n_act = 0;
            for (int a = 0; a < A; ++a) {
                const int ea = expert_of[a];
                cnt += ea == tid ? 1 : 0;
                off += ea < tid ? 1 : 0;
                arank += (flag[a] && ea < tid) ? 1 : 0;  // activated experts below this one
                n_act += flag[a];
            }
            if (tid < E) {
                counts[tid] = cnt;
                offsets[tid] = off;
                if (tid >= n_act)
                    active[tid] = -1;
                if (cnt > 0) {
                    active[arank] = tid;
                    if (plan.header != nullptr) {  // one segment and one pair per activated expert
                        Segment sg;
                        sg.expert = tid;
                        sg.row0 = off;
                        sg.n = cnt;
                        sg.first_seg = arank;
                        plan.seg[arank] = sg;
                        plan.done_routed[arank] = 0;
                        PairEntry pe;
                        pe.expert = tid;
                        pe.row0 = off;
                        pe.n = cnt;
                        pe.first_seg = arank;
                        pe.seg = arank;
                        pe.pad[0] = pe.pad[1] = pe.pad[2] = 0;
                        plan.pairs[arank] = pe;
                    }
                }
            }
            if (tid == 0) {
                offsets[E] = A;
                n_active[0] = n_act;
                if (plan.header != nullptr) {
                    plan.header[0] = n_act;  // segments
                    plan.header[1] = n_act;  // pairs
                    plan.header[2] = 0;
                    plan.header[3] = 0;
                }
            }
        } else if (blockIdx.x >= 2) {
            const int vec_per_row = H >> 3;
            const int n_copy = gridDim.x - 2;
            for (int r = blockIdx.x - 2; r < A; r += n_copy) {
                const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)token_of[r] * H);
                uint4 *dst = reinterpret_cast<uint4 *>(x_sorted + (size_t)r * H);
                for (int v = tid; v < vec_per_row; v += PERM_THREADS)
                    dst[v] = src[v];
            }
        }
        return;
    }

    // counting sort, one assignment per thread (threads beyond A idle along)
    const bool few = E <= 32;
    const int my_e = tid < A ? expert_of[tid] : -1;
    const bool my_valid = my_e >= 0 && my_e < E;
    warp_histogram_add(hist, my_e, my_valid, few);
    const uint32_t peers = __match_any_sync(0xffffffffu, my_valid ? my_e : -1);
    const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
    if (my_valid && lane == __ffs(peers) - 1)
        wcount[warp][my_e] = (uint16_t)__popc(peers);
    __syncthreads();
    if (tid < MOE_MAX_EXPERTS)
        offs[tid] = tid < E ? hist[tid] : 0;
    __syncthreads();
    block_exclusive_scan(offs, tmp, E, &total);
    int pos = 0;
    if (my_valid) {
        pos = offs[my_e] + rank_in_warp;
        for (int w = 0; w < warp; ++w)
            pos += wcount[w][my_e];
    }

    if (blockIdx.x == 0) {
        if (my_valid) {
            perm[pos] = tid;
            inv_perm[tid] = pos;
        }
    } else if (blockIdx.x == 1) {
        write_tables(hist, offs, flag, tmp, &total, E, counts, offsets, active, n_active, status, plan);
    } else {
        if (my_valid)
            token_of[pos] = tid / k;
        __syncthreads();
        const int vec_per_row = H >> 3;
        const int n_copy = gridDim.x - 2;
        for (int r = blockIdx.x - 2; r < A; r += n_copy) {
            const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)token_of[r] * H);
            uint4 *dst = reinterpret_cast<uint4 *>(x_sorted + (size_t)r * H);
            for (int v = tid; v < vec_per_row; v += PERM_THREADS)
                dst[v] = src[v];
        }
    }
}

bool route_group_small_applies(const moe_config_t &c, int T)
{
    return T <= ROUTE_SMALL_TOKENS && T * c.top_k <= ROUTE_SMALL_ASSIGN;
}

cudaError_t launch_route_group_small(const moe_config_t &c, const float *logits,
                                     const __nv_bfloat16 *x, int T, int32_t *topk_idx, float *topk_w,
                                     int32_t *counts, int32_t *offsets, int32_t *perm,
                                     int32_t *inv_perm, int32_t *active, int32_t *n_active,
                                     int32_t *status, PlanView plan, __nv_bfloat16 *x_sorted,
                                     cudaStream_t s)
{
    if (!route_group_small_applies(c, T))
        return cudaErrorInvalidValue;
    const int A = T * c.top_k, E = c.n_experts;
    // copy CTAs: one per sorted row up to 64 (a CTA moves a row of H values in one or two steps)
    const int blocks = 2 + (A < 64 ? A : 64);
#define MOE_RG_LAUNCH(V)                                                                         \
    err = launch_pdl(route_group_small_kernel<V>, dim3(blocks), dim3(PERM_THREADS), 0, s, logits, \
                     x, T, c.hidden, E, c.top_k, c.score_fn, c.renormalize, c.routed_scale,       \
                     topk_idx, topk_w, counts, offsets, perm, inv_perm, active, n_active, status, \
                     plan, x_sorted)
    cudaError_t err = cudaSuccess;
    if (E <= 32)
        MOE_RG_LAUNCH(1);
    else if (E <= 64)
        MOE_RG_LAUNCH(2);
    else if (E <= 128)
        MOE_RG_LAUNCH(4);
    else if (E <= 256)
        MOE_RG_LAUNCH(8);
    else
        MOE_RG_LAUNCH(16);
#undef MOE_RG_LAUNCH
    return err;
}

// Stand-alone plan (moe_grouped_swiglu gets its offsets from the caller).
__global__ void __launch_bounds__(MOE_MAX_EXPERTS)
plan_kernel(const int32_t *__restrict__ offsets, int E, int T, int32_t *__restrict__ status, PlanView plan)
{
    __shared__ int cnt[MOE_MAX_EXPERTS];
    __shared__ int offs[MOE_MAX_EXPERTS];
    __shared__ int scan[MOE_MAX_EXPERTS];
    __shared__ int tmp[MOE_MAX_EXPERTS];
    __shared__ int total;
    griddep_wait();
    // first kernel of the stand-alone FFN call: the shared expert's progress counters must be
    // clear before the gate/up pass, which may start right away, counts on them
    for (int i = threadIdx.x; i < max_shared_segments(T); i += blockDim.x)
        plan.done_shared[i] = 0;
    if (threadIdx.x == 0)
        status_region_init(status);
    __threadfence();
    __syncthreads();
    griddep_launch();
    const int tid = threadIdx.x;
    int row0 = 0, n = 0;
    if (tid < E) {
        row0 = offsets[tid];
        n = offsets[tid + 1] - row0;
    }
    cnt[tid] = n;
    offs[tid] = row0;
    __syncthreads();
    build_plan(cnt, offs, scan, tmp, &total, E, status, plan);
}

cudaError_t launch_plan(const moe_config_t &c, int T, const int32_t *offsets, int32_t *status,
                        PlanView plan, cudaStream_t s)
{
    return launch_pdl(plan_kernel, dim3(1), dim3(MOE_MAX_EXPERTS), 0, s, offsets, c.n_experts, T, status,
                      plan);
}

}  // namespace moe

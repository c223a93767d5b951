// The whole layer for a handful of tokens in ONE launch (moe_verify_layer with T <= 4).
//
// With one to four tokens every activated expert sees one to four rows (Eq. T_exp: about one),
// so the layer is a stream of weight rows against a few vectors: Sec. 3.3's "the cost is loading
// the activated experts" in its purest form.  A chain of kernels pays a launch boundary and a
// pipeline fill per step, which at this size costs more than the weights take to load.  Here one
// cooperative grid (one CTA per SM) walks the steps with grid-wide barriers in between:
//
//   A  partial router logits (router rows cut into column chunks, one warp each) and, since it
//      does not depend on the routing, the shared expert's gate/up projection + SwiGLU
//   -- barrier --  every CTA sums the partial logits, selects the top-k experts and groups the
//      assignments for itself (a few hundred values); CTA 0 writes the routing tables out
//   B  gate/up projection + SwiGLU of the activated experts' rows
//   -- barrier --
//   C  down projection of every group and of the shared expert, cut into column chunks; partial
//      sums in fp32
//   -- barrier --
//   D  gate-weighted combine of the partial sums, rounded once to bf16
//
// The projections run on the CUDA cores: a warp takes four weight rows at a time, every lane
// 16-byte pieces of them (streamed past L1), and multiplies them with the group's token rows,
// which it re-reads through L1.  Four weight rows share each token value a lane loads and keep
// eight to sixteen 16-byte loads per lane in flight.
#include <stdlib.h>

#include <atomic>

#include "common.cuh"
#include "route_topk.cuh"

namespace moe {

constexpr int LS_THREADS = 512;
constexpr int LS_WARPS = LS_THREADS / 32;
constexpr int LS_MAX_TOKENS = 4;     // rows a warp carries per weight row (accumulators in registers)
constexpr int LS_MAX_ASSIGN = 32;    // T * top_k: one warp sorts the assignments
constexpr int LS_LOGIT_CHUNK = 512;  // router-row columns per work item
constexpr int LS_DOWN_CHUNK = 2048;  // most columns of a down-projection work item
constexpr uint64_t LS_WAIT_NS = 1000ull * 1000ull * 1000ull;
constexpr int LS_BARRIER_WORD = 8;  // int32 index inside the status region of the three barrier words

struct SmallArgs {
    int T, H, E, K, I, Is;
    int score_fn, renormalize, gated;
    float routed_scale;
    const float *w_router, *router_bias;
    const __nv_bfloat16 *w_gate, *w_up, *w_down, *ws_gate, *ws_up, *ws_down, *w_shared_gate;
    const __nv_bfloat16 *x;
    __nv_bfloat16 *out;
    // workspace
    float *logit_part;  // [E (+1), logit chunks, LS_MAX_TOKENS]
    float *logits, *topk_w, *shared_scale;
    int32_t *topk_idx, *counts, *offsets, *active, *n_active, *perm, *inv_perm;
    __nv_bfloat16 *h, *h_shared;
    float *y_part;                // routed [chunks_r, A, H] then shared [chunks_s, T, H]
    unsigned long long *barrier;  // three words, one per barrier: (epoch << 32) | arrivals
    int32_t *status;
    uint32_t epoch;
    int wait_us;
    int logit_chunks;       // ceil(H / LS_LOGIT_CHUNK)
    int chunk_r, chunks_r;  // columns per down-projection chunk of a routed group, their number
    int chunk_s, chunks_s;  // the same for the shared expert
};

// ---- loads ---------------------------------------------------------------------------------

// weights: read once by one lane of the whole grid
__device__ __forceinline__ uint4 ld_stream_16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void unpack8(const uint4 v, float (&f)[8])
{
    f[0] = bf16_lo(v.x);
    f[1] = bf16_hi(v.x);
    f[2] = bf16_lo(v.y);
    f[3] = bf16_hi(v.y);
    f[4] = bf16_lo(v.z);
    f[5] = bf16_hi(v.z);
    f[6] = bf16_lo(v.w);
    f[7] = bf16_hi(v.w);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// ---- four weight rows against NR token rows ---------------------------------------------------
//
// acc[j][r] = sum over columns [0, ncols) of w[j][col] * xr[r][col], j < 4, r < NR, summed over
// the warp's lanes on return (every lane holds the totals).  ncols is a multiple of 8; w[j] and
// xr[r] are 16-byte aligned.  A step covers 512 columns: lane l takes columns 8 l .. 8 l + 7 of
// each half, so a warp reads 512 contiguous bytes of a row per load.  The loads of the next step
// are issued before the arithmetic of the current one.
template <int NR>
__device__ __forceinline__ void rows4_dot(const __nv_bfloat16 *const (&w)[4], int ncols,
                                          const __nv_bfloat16 *const (&xr)[NR], int lane,
                                          float (&acc)[4][NR])
{
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int r = 0; r < NR; ++r)
            acc[j][r] = 0.f;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    uint4 cur[8];
    {
        const int c0 = lane * 8, c1 = 256 + lane * 8;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            cur[2 * j] = c0 < ncols ? ld_stream_16(w[j] + c0) : zero;
            cur[2 * j + 1] = c1 < ncols ? ld_stream_16(w[j] + c1) : zero;
        }
    }
#pragma unroll 1
    for (int base = 0; base < ncols; base += 512) {
        uint4 nxt[8];
        {
            const int c0 = base + 512 + lane * 8, c1 = c0 + 256;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                nxt[2 * j] = c0 < ncols ? ld_stream_16(w[j] + c0) : zero;
                nxt[2 * j + 1] = c1 < ncols ? ld_stream_16(w[j] + c1) : zero;
            }
        }
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int col = base + half * 256 + lane * 8;
            if (col < ncols) {
                float xf[NR][8];
#pragma unroll
                for (int r = 0; r < NR; ++r)
                    unpack8(ld_cached_v4(xr[r] + col), xf[r]);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float wf[8];
                    unpack8(cur[2 * j + half], wf);
#pragma unroll
                    for (int r = 0; r < NR; ++r)
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            acc[j][r] = fmaf(wf[q], xf[r][q], acc[j][r]);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 8; ++q)
            cur[q] = nxt[q];
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int r = 0; r < NR; ++r)
            acc[j][r] = warp_sum(acc[j][r]);
}

// Gate/up + SwiGLU of two intermediate features i0, i0 + 1 for NR rows:
// h[r][i] = bf16( silu(Wg[i,:] . x[r,:]) * (Wu[i,:] . x[r,:]) ).
template <int NR>
__device__ __forceinline__ void gateup_item(const __nv_bfloat16 *wg, const __nv_bfloat16 *wu, int H,
                                            int i0, const __nv_bfloat16 *const (&xr)[NR],
                                            __nv_bfloat16 *const (&hr)[NR], int lane)
{
    const __nv_bfloat16 *const w[4] = {wg + (size_t)i0 * H, wg + (size_t)(i0 + 1) * H,
                                      wu + (size_t)i0 * H, wu + (size_t)(i0 + 1) * H};
    float acc[4][NR];
    rows4_dot<NR>(w, H, xr, lane, acc);
    if (lane == 0) {
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            const float h0 = silu_f(acc[0][r]) * acc[2][r];
            const float h1 = silu_f(acc[1][r]) * acc[3][r];
            *reinterpret_cast<__nv_bfloat162 *>(hr[r] + i0) = __floats2bfloat162_rn(h0, h1);
        }
    }
}

// Down projection of four output features f0 .. f0 + 3 over the columns [c0, c0 + ncols) of the
// intermediate for NR rows; the partial sums go to yp[r][f0 .. f0 + 3] (fp32).
template <int NR>
__device__ __forceinline__ void down_item(const __nv_bfloat16 *wd, int ld, int f0, int c0, int ncols,
                                          const __nv_bfloat16 *const (&hr)[NR],
                                          float *const (&yp)[NR], int lane)
{
    const __nv_bfloat16 *const w[4] = {wd + (size_t)f0 * ld + c0, wd + (size_t)(f0 + 1) * ld + c0,
                                      wd + (size_t)(f0 + 2) * ld + c0,
                                      wd + (size_t)(f0 + 3) * ld + c0};
    const __nv_bfloat16 *hc[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r)
        hc[r] = hr[r] + c0;
    float acc[4][NR];
    rows4_dot<NR>(w, ncols, hc, lane, acc);
    if (lane == 0) {
#pragma unroll
        for (int r = 0; r < NR; ++r)
            *reinterpret_cast<float4 *>(yp[r] + f0) =
                make_float4(acc[0][r], acc[1][r], acc[2][r], acc[3][r]);
    }
}

// ---- grid barrier -----------------------------------------------------------------------------
//
// One 64-bit word per barrier: the call's epoch in the high half, the number of CTAs that have
// arrived in the low half.  The workspace need not be initialised and may hold the word of an
// earlier call (complete or abandoned): the first CTA to arrive finds another epoch there and
// replaces the word by (epoch, 0) before anybody adds to it.  Every CTA of the cooperative grid is
// resident, so all arrive; the wait is bounded all the same and raises the status word when it
// gives up.  Returns false then, and the CTA leaves the kernel.
__device__ __forceinline__ bool grid_barrier(unsigned long long *word, uint32_t epoch,
                                             uint32_t n_ctas, int32_t *status, int wait_us,
                                             int *s_ok)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();  // this CTA's stores (ordered before by the barrier above) become visible
        const unsigned long long base = (unsigned long long)epoch << 32;
        unsigned long long seen = *reinterpret_cast<volatile unsigned long long *>(word);
        while ((uint32_t)(seen >> 32) != epoch) {
            const unsigned long long prev = atomicCAS(word, seen, base);
            if (prev == seen)
                break;
            seen = prev;
        }
        atomicAdd(word, 1ull);
        const unsigned long long target = base + n_ctas;
        auto reached = [&]() {
            unsigned long long v;
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
            return v == target;
        };
        bool ok = reached();
        if (!ok) {
            uint64_t t0;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
            for (;;) {
#pragma unroll 1
                for (int i = 0; i < 32 && !ok; ++i) {
                    ok = reached();
                    if (!ok)
                        __nanosleep(40);
                }
                if (ok)
                    break;
                uint64_t t1;
                asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
                if (t1 - t0 > 1000ull * (uint64_t)wait_us) {
                    atomicExch(status, 1);
                    break;
                }
            }
        }
        *s_ok = ok ? 1 : 0;
    }
    __syncthreads();
    return *s_ok != 0;
}

// ---- the kernel -------------------------------------------------------------------------------

template <int VPL>
__global__ void __launch_bounds__(LS_THREADS, 1) layer_small_kernel(const SmallArgs a)
{
    __shared__ float s_z[LS_MAX_TOKENS][MOE_MAX_EXPERTS];  // logits of the call's tokens
    __shared__ float s_gate_w[LS_MAX_ASSIGN];              // by assignment t * K + j
    __shared__ int s_expert_of[LS_MAX_ASSIGN];             // by assignment
    __shared__ int s_pos_of[LS_MAX_ASSIGN];                // sorted row of an assignment
    __shared__ int s_token_of[LS_MAX_ASSIGN];              // by sorted row
    __shared__ int s_leader[LS_MAX_ASSIGN];                // assignment is the first of its expert
    __shared__ int s_grp_expert[LS_MAX_ASSIGN], s_grp_row0[LS_MAX_ASSIGN], s_grp_n[LS_MAX_ASSIGN];
    __shared__ float s_shared_scale[LS_MAX_TOKENS];
    __shared__ int s_n_groups;
    __shared__ int s_ok;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x;
    const int n_warps = G * LS_WARPS;
    const int gwarp = warp * G + blockIdx.x;  // consecutive work items land on different SMs
    const int T = a.T, H = a.H, E = a.E, K = a.K, A = a.T * a.K;

    if (blockIdx.x == 0 && tid == 0)
        status_region_init(a.status);

    // ---- A: partial logits, shared expert's gate/up ---------------------------------------------
    {
        const int rows = E + (a.gated ? 1 : 0);
        const int n_logit = rows * a.logit_chunks;
        const int n_shared = a.Is >> 1;
        for (int item = gwarp; item < n_logit + n_shared; item += n_warps) {
            if (item < n_logit) {
                const int r = item / a.logit_chunks, c = item - r * a.logit_chunks;
                const int col0 = c * LS_LOGIT_CHUNK;
                float acc[LS_MAX_TOKENS] = {0.f, 0.f, 0.f, 0.f};
                if (r < E) {
                    const float *wr = a.w_router + (size_t)r * H;
                    float4 wv[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int col = col0 + q * 128 + lane * 4;
                        wv[q] = col < H ? __ldg(reinterpret_cast<const float4 *>(wr + col))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int col = col0 + q * 128 + lane * 4;
                        if (col < H) {
#pragma unroll
                            for (int t = 0; t < LS_MAX_TOKENS; ++t) {
                                if (t < T) {
                                    const uint2 xv = __ldg(reinterpret_cast<const uint2 *>(
                                        a.x + (size_t)t * H + col));
                                    acc[t] = fmaf(wv[q].x, bf16_lo(xv.x), acc[t]);
                                    acc[t] = fmaf(wv[q].y, bf16_hi(xv.x), acc[t]);
                                    acc[t] = fmaf(wv[q].z, bf16_lo(xv.y), acc[t]);
                                    acc[t] = fmaf(wv[q].w, bf16_hi(xv.y), acc[t]);
                                }
                            }
                        }
                    }
                } else {  // the shared expert's gate row (bf16)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int col = col0 + q * 128 + lane * 4;
                        if (col < H) {
                            const uint2 wv =
                                __ldg(reinterpret_cast<const uint2 *>(a.w_shared_gate + col));
#pragma unroll
                            for (int t = 0; t < LS_MAX_TOKENS; ++t) {
                                if (t < T) {
                                    const uint2 xv = __ldg(reinterpret_cast<const uint2 *>(
                                        a.x + (size_t)t * H + col));
                                    acc[t] = fmaf(bf16_lo(wv.x), bf16_lo(xv.x), acc[t]);
                                    acc[t] = fmaf(bf16_hi(wv.x), bf16_hi(xv.x), acc[t]);
                                    acc[t] = fmaf(bf16_lo(wv.y), bf16_lo(xv.y), acc[t]);
                                    acc[t] = fmaf(bf16_hi(wv.y), bf16_hi(xv.y), acc[t]);
                                }
                            }
                        }
                    }
                }
#pragma unroll
                for (int t = 0; t < LS_MAX_TOKENS; ++t)
                    acc[t] = warp_sum(acc[t]);
                if (lane == 0)
                    *reinterpret_cast<float4 *>(a.logit_part + (size_t)item * LS_MAX_TOKENS) =
                        make_float4(acc[0], acc[1], acc[2], acc[3]);
            } else {
                const int i0 = (item - n_logit) * 2;
#define LS_SHARED_GATEUP(NR)                                                             \
    {                                                                                    \
        const __nv_bfloat16 *xr[NR];                                                     \
        __nv_bfloat16 *hr[NR];                                                           \
        _Pragma("unroll") for (int r = 0; r < NR; ++r)                                   \
        {                                                                                \
            xr[r] = a.x + (size_t)r * H;                                                 \
            hr[r] = a.h_shared + (size_t)r * a.Is;                                       \
        }                                                                                \
        gateup_item<NR>(a.ws_gate, a.ws_up, H, i0, xr, hr, lane);                        \
    }
                switch (T) {
                case 1: LS_SHARED_GATEUP(1) break;
                case 2: LS_SHARED_GATEUP(2) break;
                case 3: LS_SHARED_GATEUP(3) break;
                default: LS_SHARED_GATEUP(4) break;
                }
#undef LS_SHARED_GATEUP
            }
        }
    }
    if (!grid_barrier(a.barrier + 0, a.epoch, G, a.status, a.wait_us, &s_ok))
        return;

    // ---- routing: every CTA for itself ----------------------------------------------------------
    if (warp < T) {
        const int t = warp;
        for (int e = lane; e < E; e += 32) {
            float z = 0.f;
            const float *p = a.logit_part + (size_t)e * a.logit_chunks * LS_MAX_TOKENS + t;
            for (int c = 0; c < a.logit_chunks; ++c)
                z += __ldcg(p + c * LS_MAX_TOKENS);
            if (a.router_bias != nullptr)
                z += a.router_bias[e];
            s_z[t][e] = z;
            if (blockIdx.x == 0)
                a.logits[(size_t)t * E + e] = z;
        }
        if (a.gated && lane == 0) {
            float z = 0.f;
            const float *p = a.logit_part + (size_t)E * a.logit_chunks * LS_MAX_TOKENS + t;
            for (int c = 0; c < a.logit_chunks; ++c)
                z += __ldcg(p + c * LS_MAX_TOKENS);
            const float sc = 1.0f / (1.0f + expf(-z));
            s_shared_scale[t] = sc;
            if (blockIdx.x == 0)
                a.shared_scale[t] = sc;
        }
        __syncwarp();
        int sel_i;
        float sel_w;
        warp_route_topk<VPL>(s_z[t], E, K, a.score_fn, a.renormalize, a.routed_scale, lane, sel_i,
                             sel_w);
        if (lane < K) {
            s_expert_of[t * K + lane] = sel_i;
            s_gate_w[t * K + lane] = sel_w;
            if (blockIdx.x == 0) {
                a.topk_idx[t * K + lane] = sel_i;
                a.topk_w[t * K + lane] = sel_w;
            }
        }
    }
    __syncthreads();
    if (warp == 0) {
        // stable sort of at most 32 assignments by expert, groups in ascending expert order
        const int e = lane < A ? s_expert_of[lane] : -1;
        const uint32_t peers = __match_any_sync(0xffffffffu, e);
        const int rank = __popc(peers & ((1u << lane) - 1u));
        const bool leader = e >= 0 && lane == __ffs(peers) - 1;
        int less = 0, groups_below = 0;
#pragma unroll
        for (int src = 0; src < 32; ++src) {
            const int other = __shfl_sync(0xffffffffu, e, src);
            const int other_leads = __shfl_sync(0xffffffffu, leader ? 1 : 0, src);
            const bool below = other >= 0 && other < e;
            less += below ? 1 : 0;
            groups_below += (below && other_leads) ? 1 : 0;
        }
        const uint32_t leaders = __ballot_sync(0xffffffffu, leader);
        s_leader[lane] = leader ? 1 : 0;
        if (e >= 0) {
            const int pos = less + rank;
            s_pos_of[lane] = pos;
            s_token_of[pos] = lane / K;
            if (leader) {
                s_grp_expert[groups_below] = e;
                s_grp_row0[groups_below] = less;
                s_grp_n[groups_below] = __popc(peers);
            }
            if (blockIdx.x == 0) {
                a.perm[pos] = lane;
                a.inv_perm[lane] = pos;
            }
        }
        if (lane == 0)
            s_n_groups = __popc(leaders);
    }
    __syncthreads();
    if (blockIdx.x == 0) {
        // routing tables (copies for the caller; the kernel itself works from shared memory)
        for (int e = tid; e < E; e += LS_THREADS) {
            int cnt = 0, off = 0, arank = 0;
            for (int i = 0; i < A; ++i) {
                const int ea = s_expert_of[i];
                cnt += ea == e ? 1 : 0;
                off += ea < e ? 1 : 0;
                arank += (s_leader[i] && ea < e) ? 1 : 0;
            }
            a.counts[e] = cnt;
            a.offsets[e] = off;
            if (e >= s_n_groups)
                a.active[e] = -1;
            if (cnt > 0)
                a.active[arank] = e;
        }
        if (tid == 0) {
            a.offsets[E] = A;
            a.n_active[0] = s_n_groups;
        }
    }

    // ---- B: gate/up + SwiGLU of the activated experts ----------------------------------------
    {
        const int per_group = a.I >> 1;
        const int n_items = s_n_groups * per_group;
        for (int item = gwarp; item < n_items; item += n_warps) {
            const int g = item / per_group, i0 = (item - g * per_group) * 2;
            const int e = s_grp_expert[g], row0 = s_grp_row0[g], n = s_grp_n[g];
            const __nv_bfloat16 *wg = a.w_gate + (size_t)e * a.I * H;
            const __nv_bfloat16 *wu = a.w_up + (size_t)e * a.I * H;
#define LS_ROUTED_GATEUP(NR)                                                             \
    {                                                                                    \
        const __nv_bfloat16 *xr[NR];                                                     \
        __nv_bfloat16 *hr[NR];                                                           \
        _Pragma("unroll") for (int r = 0; r < NR; ++r)                                   \
        {                                                                                \
            xr[r] = a.x + (size_t)s_token_of[row0 + r] * H;                              \
            hr[r] = a.h + (size_t)(row0 + r) * a.I;                                      \
        }                                                                                \
        gateup_item<NR>(wg, wu, H, i0, xr, hr, lane);                                    \
    }
            switch (n) {
            case 1: LS_ROUTED_GATEUP(1) break;
            case 2: LS_ROUTED_GATEUP(2) break;
            case 3: LS_ROUTED_GATEUP(3) break;
            default: LS_ROUTED_GATEUP(4) break;
            }
#undef LS_ROUTED_GATEUP
        }
    }
    if (!grid_barrier(a.barrier + 1, a.epoch, G, a.status, a.wait_us, &s_ok))
        return;

    // ---- C: down projection, partial sums per column chunk ---------------------------------------
    {
        const int f_items = H >> 2;
        const int per_group = a.chunks_r * f_items;
        const int n_routed = s_n_groups * per_group;
        const int n_shared = a.chunks_s * f_items;
        float *yp_shared = a.y_part + (size_t)a.chunks_r * A * H;
        for (int item = gwarp; item < n_routed + n_shared; item += n_warps) {
            if (item < n_routed) {
                const int g = item / per_group;
                const int rem = item - g * per_group;
                const int c = rem / f_items, f0 = (rem - c * f_items) * 4;
                const int e = s_grp_expert[g], row0 = s_grp_row0[g], n = s_grp_n[g];
                const int c0 = c * a.chunk_r;
                const int ncols = min(a.chunk_r, a.I - c0);
                const __nv_bfloat16 *wd = a.w_down + (size_t)e * H * a.I;
#define LS_ROUTED_DOWN(NR)                                                               \
    {                                                                                    \
        const __nv_bfloat16 *hr[NR];                                                     \
        float *yp[NR];                                                                   \
        _Pragma("unroll") for (int r = 0; r < NR; ++r)                                   \
        {                                                                                \
            hr[r] = a.h + (size_t)(row0 + r) * a.I;                                      \
            yp[r] = a.y_part + ((size_t)c * A + row0 + r) * H;                           \
        }                                                                                \
        down_item<NR>(wd, a.I, f0, c0, ncols, hr, yp, lane);                             \
    }
                switch (n) {
                case 1: LS_ROUTED_DOWN(1) break;
                case 2: LS_ROUTED_DOWN(2) break;
                case 3: LS_ROUTED_DOWN(3) break;
                default: LS_ROUTED_DOWN(4) break;
                }
#undef LS_ROUTED_DOWN
            } else {
                const int rem = item - n_routed;
                const int c = rem / f_items, f0 = (rem - c * f_items) * 4;
                const int c0 = c * a.chunk_s;
                const int ncols = min(a.chunk_s, a.Is - c0);
#define LS_SHARED_DOWN(NR)                                                               \
    {                                                                                    \
        const __nv_bfloat16 *hr[NR];                                                     \
        float *yp[NR];                                                                   \
        _Pragma("unroll") for (int r = 0; r < NR; ++r)                                   \
        {                                                                                \
            hr[r] = a.h_shared + (size_t)r * a.Is;                                       \
            yp[r] = yp_shared + ((size_t)c * T + r) * H;                                 \
        }                                                                                \
        down_item<NR>(a.ws_down, a.Is, f0, c0, ncols, hr, yp, lane);                     \
    }
                switch (T) {
                case 1: LS_SHARED_DOWN(1) break;
                case 2: LS_SHARED_DOWN(2) break;
                case 3: LS_SHARED_DOWN(3) break;
                default: LS_SHARED_DOWN(4) break;
                }
#undef LS_SHARED_DOWN
            }
        }
    }
    if (!grid_barrier(a.barrier + 2, a.epoch, G, a.status, a.wait_us, &s_ok))
        return;

    // ---- D: combine -------------------------------------------------------------------------------
    {
        const int f_vec = H >> 2;
        const float *yp_shared = a.y_part + (size_t)a.chunks_r * A * H;
        for (int v = blockIdx.x * LS_THREADS + tid; v < T * f_vec; v += G * LS_THREADS) {
            const int t = v / f_vec, f = (v - t * f_vec) * 4;
            float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int j = 0; j < K; ++j) {
                const int row = s_pos_of[t * K + j];
                float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int c = 0; c < a.chunks_r; ++c) {
                    const float4 p = __ldcg(reinterpret_cast<const float4 *>(
                        a.y_part + ((size_t)c * A + row) * H + f));
                    y.x += p.x;
                    y.y += p.y;
                    y.z += p.z;
                    y.w += p.w;
                }
                const float gw = s_gate_w[t * K + j];
                o.x = fmaf(gw, y.x, o.x);
                o.y = fmaf(gw, y.y, o.y);
                o.z = fmaf(gw, y.z, o.z);
                o.w = fmaf(gw, y.w, o.w);
            }
            if (a.Is > 0) {
                float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int c = 0; c < a.chunks_s; ++c) {
                    const float4 p = __ldcg(reinterpret_cast<const float4 *>(
                        yp_shared + ((size_t)c * T + t) * H + f));
                    y.x += p.x;
                    y.y += p.y;
                    y.z += p.z;
                    y.w += p.w;
                }
                const float sc = a.gated ? s_shared_scale[t] : 1.0f;
                o.x = fmaf(sc, y.x, o.x);
                o.y = fmaf(sc, y.y, o.y);
                o.z = fmaf(sc, y.z, o.z);
                o.w = fmaf(sc, y.w, o.w);
            }
            const __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y);
            const __nv_bfloat162 hi = __floats2bfloat162_rn(o.z, o.w);
            uint2 packed;
            packed.x = *reinterpret_cast<const uint32_t *>(&lo);
            packed.y = *reinterpret_cast<const uint32_t *>(&hi);
            *reinterpret_cast<uint2 *>(a.out + (size_t)t * H + f) = packed;
        }
    }
}

// ---- host -------------------------------------------------------------------------------------

static int down_chunks(int cols) { return (cols + LS_DOWN_CHUNK - 1) / LS_DOWN_CHUNK; }

// columns per chunk: equal shares, rounded up to a whole half-step of the row walk
static int down_chunk_cols(int cols)
{
    const int n = down_chunks(cols);
    return n == 0 ? 0 : (((cols + n - 1) / n) + 255) & ~255;
}

static bool small_shape(const moe_config_t &c, int T)
{
    return T <= LS_MAX_TOKENS && T * c.top_k <= LS_MAX_ASSIGN;
}

size_t layer_small_logit_part_bytes(const moe_config_t &c)
{
    const size_t chunks = (c.hidden + LS_LOGIT_CHUNK - 1) / LS_LOGIT_CHUNK;
    return ((size_t)c.n_experts + 1) * chunks * LS_MAX_TOKENS * sizeof(float);
}

size_t layer_small_y_part_bytes(const moe_config_t &c, int T)
{
    // sized for the largest small call, so that the layout never shrinks as T grows
    int t = T < LS_MAX_TOKENS ? T : LS_MAX_TOKENS;
    while (t > 0 && !small_shape(c, t))
        --t;
    if (t == 0)
        return 0;
    const size_t rows =
        (size_t)down_chunks(c.inter) * t * c.top_k + (size_t)down_chunks(c.shared_inter) * t;
    return rows * c.hidden * sizeof(float);
}

int small_layer_override()
{
    static const int v = [] {
        const char *e = getenv("MOE_SMALL_FUSED");
        return !e ? -1 : (e[0] == '0' ? 0 : -1);
    }();
    return v;
}

static bool cooperative_ok()
{
    static int cached[MAX_DEVICE_ORDINALS];  // 0 unknown, 1 yes, -1 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICE_ORDINALS)
        return false;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess)
            v = 0;
        cached[dev] = v ? 1 : -1;
    }
    return cached[dev] == 1;
}

bool layer_small_applies(const moe_config_t &c, int T)
{
    return small_shape(c, T) && small_layer_override() != 0 && cooperative_ok();
}

cudaError_t launch_layer_small(const moe_config_t &c, const moe_weights_t &w, const __nv_bfloat16 *x,
                               int T, __nv_bfloat16 *out, char *ws, const Workspace &L,
                               cudaStream_t s)
{
    if (!layer_small_applies(c, T))
        return cudaErrorInvalidValue;
    static std::atomic<uint32_t> next_epoch{1};
    uint32_t epoch = next_epoch.fetch_add(1, std::memory_order_relaxed);
    if (epoch == 0)
        epoch = next_epoch.fetch_add(1, std::memory_order_relaxed);
    SmallArgs a{};
    a.T = T;
    a.H = c.hidden;
    a.E = c.n_experts;
    a.K = c.top_k;
    a.I = c.inter;
    a.Is = c.shared_inter;
    a.score_fn = c.score_fn;
    a.renormalize = c.renormalize;
    a.gated = (c.shared_inter > 0 && c.shared_gate) ? 1 : 0;
    a.routed_scale = c.routed_scale;
    a.w_router = w.w_router;
    a.router_bias = w.router_bias;
    a.w_gate = static_cast<const __nv_bfloat16 *>(w.w_gate);
    a.w_up = static_cast<const __nv_bfloat16 *>(w.w_up);
    a.w_down = static_cast<const __nv_bfloat16 *>(w.w_down);
    a.ws_gate = static_cast<const __nv_bfloat16 *>(w.ws_gate);
    a.ws_up = static_cast<const __nv_bfloat16 *>(w.ws_up);
    a.ws_down = static_cast<const __nv_bfloat16 *>(w.ws_down);
    a.w_shared_gate = static_cast<const __nv_bfloat16 *>(w.w_shared_gate);
    a.x = x;
    a.out = out;
    a.logit_part = reinterpret_cast<float *>(ws + L.small_logit_part);
    a.logits = reinterpret_cast<float *>(ws + L.logits);
    a.topk_w = reinterpret_cast<float *>(ws + L.topk_w);
    a.shared_scale = reinterpret_cast<float *>(ws + L.shared_scale);
    a.topk_idx = reinterpret_cast<int32_t *>(ws + L.topk_idx);
    a.counts = reinterpret_cast<int32_t *>(ws + L.counts);
    a.offsets = reinterpret_cast<int32_t *>(ws + L.offsets);
    a.active = reinterpret_cast<int32_t *>(ws + L.active);
    a.n_active = reinterpret_cast<int32_t *>(ws + L.n_active);
    a.perm = reinterpret_cast<int32_t *>(ws + L.perm);
    a.inv_perm = reinterpret_cast<int32_t *>(ws + L.inv_perm);
    a.h = reinterpret_cast<__nv_bfloat16 *>(ws + L.h);
    a.h_shared = reinterpret_cast<__nv_bfloat16 *>(ws + L.h_shared);
    a.y_part = reinterpret_cast<float *>(ws + L.small_y_part);
    a.status = reinterpret_cast<int32_t *>(ws + L.status);
    a.barrier = reinterpret_cast<unsigned long long *>(a.status + LS_BARRIER_WORD);
    a.epoch = epoch;
    a.wait_us = (int)(LS_WAIT_NS / 1000ull);
    a.logit_chunks = (c.hidden + LS_LOGIT_CHUNK - 1) / LS_LOGIT_CHUNK;
    a.chunks_r = down_chunks(c.inter);
    a.chunk_r = down_chunk_cols(c.inter);
    a.chunks_s = down_chunks(c.shared_inter);
    a.chunk_s = down_chunk_cols(c.shared_inter);

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(sm_count());
    cfg.blockDim = dim3(LS_THREADS);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int E = c.n_experts;
    if (E <= 32)
        return cudaLaunchKernelEx(&cfg, layer_small_kernel<1>, a);
    if (E <= 64)
        return cudaLaunchKernelEx(&cfg, layer_small_kernel<2>, a);
    if (E <= 128)
        return cudaLaunchKernelEx(&cfg, layer_small_kernel<4>, a);
    if (E <= 256)
        return cudaLaunchKernelEx(&cfg, layer_small_kernel<8>, a);
    return cudaLaunchKernelEx(&cfg, layer_small_kernel<16>, a);
}

}  // namespace moe

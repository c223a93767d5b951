// The whole layer for a handful of tokens in ONE launch (moe_verify_layer with T <= 4).
//
// With one to four tokens every activated expert sees one to four rows (Eq. T_exp: about one),
// so the layer is a stream of weight rows against a few vectors: Sec. 3.3's "the cost is loading
// the activated experts" in its purest form.  A chain of kernels pays a launch boundary and a
// pipeline fill per step, which at this size costs more than the weights take to load.  Here one
// cooperative grid (one CTA per SM) keeps the weights streaming from the first step to the last:
//
//   1  partial router logits: router rows cut into column chunks, one warp each
//   2  four warps of every CTA wait at the kernel's only grid-wide barrier for all partial
//      logits, sum them, select the top-k experts and group the assignments -- every CTA for
//      itself, a few hundred values (CTA 0 writes the routing tables out).  The other warps
//      meanwhile stream the shared expert's gate/up projection + SwiGLU, which does not depend
//      on the routing.
//   3  gate/up projection + SwiGLU of the activated experts' rows (a "unit" is the shared expert
//      or one activated expert; work items are handed out unit by unit)
//   4  down projection: every CTA owns a few output features and computes them for every unit,
//      again unit by unit.  Before its first item of a unit a warp waits until all CTAs have
//      published that they finished the unit's gate/up items (one counter per unit): by the
//      time the last gate/up items are under way the down projection of the earlier units is
//      streaming already, so no barrier separates the two.
//   5  the CTA combines its features' partial sums with the gate weights and rounds once to bf16.
//
// The projections run on the CUDA cores: a warp takes a few weight rows at a time, every lane
// 16-byte pieces of them (streamed past L1), and multiplies them with the unit's token rows,
// which it re-reads through L1; eight 16-byte loads per lane are in flight while the previous
// eight are being consumed.
#include <stdlib.h>

#include <atomic>

#include "common.cuh"
#include "route_topk.cuh"

namespace moe {

constexpr int LS_THREADS = 512;
constexpr int LS_WARPS = LS_THREADS / 32;
constexpr int LS_MAX_TOKENS = 4;      // rows a warp carries per weight row (accumulators in registers)
constexpr int LS_MAX_ASSIGN = 32;     // T * top_k: one warp sorts the assignments
constexpr int LS_MAX_UNITS = 1 + LS_MAX_ASSIGN;  // the shared expert and the activated experts
constexpr int LS_LOGIT_CHUNK = 1024;  // router-row columns per work item
constexpr int LS_ROUTE_WARPS = 4;     // warps of every CTA that wait for the logits and do the routing
constexpr int LS_DOWN_CHUNK_MAX = 4096;  // most columns of a down-projection work item ...
constexpr int LS_DOWN_CHUNK_MIN = 2048;  // ... and the least the host goes down to for more items
constexpr int LS_DOWN_ITEMS_WANTED = 48; // down-projection items per CTA (three per warp) it aims at
constexpr size_t LS_SHARED_WORK_MAX = 80u << 20;  // T * I_s * H up to which the kernel is used for T > 1
constexpr int LS_DOWN_ROWS = 4;       // output features per down-projection work item
constexpr int LS_SLOT_FLOATS = LS_DOWN_ROWS * LS_MAX_TOKENS;  // partial sums of one such item
constexpr size_t LS_MAX_SLOT_BYTES = 160u << 10;
constexpr uint64_t LS_WAIT_NS = 1000ull * 1000ull * 1000ull;
constexpr int LS_SELFTEST_WORD = 4;  // int32 index there of the word the wait self-test waits on
constexpr int LS_BARRIER_WORD = 8;  // int32 index of the grid barrier's word inside the status region
constexpr size_t LS_UNIT_WORD_BYTES = 512;  // the units' counters lead the partial-logit region

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
    __nv_bfloat16 *h;         // [A, I_pad]: SwiGLU intermediate of the routed rows, sorted order
    __nv_bfloat16 *h_shared;  // [T, Is_pad]
    int I_pad, Is_pad;        // row pitches: whole 128-byte lines, so no line belongs to two units
    unsigned long long *barrier;    // (epoch << 32) | CTAs arrived
    unsigned long long *unit_done;  // [LS_MAX_UNITS]: (epoch << 32) | CTAs done with the unit's gate/up
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

// ---- R weight rows against NR token rows -----------------------------------------------------
//
// acc[j][r] = sum over columns [0, ncols) of w[j][col] * xr[r][col], j < R, r < NR, summed over
// the warp's lanes on return (every lane holds the totals).  ncols is a multiple of 8; w[j] and
// xr[r] are 16-byte aligned.  A step covers 8 / R parts of 256 columns: lane l takes columns
// 8 l .. 8 l + 7 of each part, so a warp reads 512 contiguous bytes of a row per load and a lane
// has eight loads per step.  The loads of the next step are issued before the arithmetic of the
// current one.
template <int R, int NR>
__device__ __forceinline__ void rows_dot(const __nv_bfloat16 *const (&w)[R], int ncols,
                                         const __nv_bfloat16 *const (&xr)[NR], int lane,
                                         float (&acc)[R][NR])
{
    constexpr int Q = 8 / R;
    constexpr int STEP = Q * 256;
#pragma unroll
    for (int j = 0; j < R; ++j)
#pragma unroll
        for (int r = 0; r < NR; ++r)
            acc[j][r] = 0.f;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    uint4 cur[8];
#pragma unroll
    for (int j = 0; j < R; ++j)
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int col = q * 256 + lane * 8;
            cur[j * Q + q] = col < ncols ? ld_stream_16(w[j] + col) : zero;
        }
#pragma unroll 1
    for (int base = 0; base < ncols; base += STEP) {
        uint4 nxt[8];
#pragma unroll
        for (int j = 0; j < R; ++j)
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                const int col = base + STEP + q * 256 + lane * 8;
                nxt[j * Q + q] = col < ncols ? ld_stream_16(w[j] + col) : zero;
            }
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int col = base + q * 256 + lane * 8;
            if (col < ncols) {
                float xf[NR][8];
#pragma unroll
                for (int r = 0; r < NR; ++r)
                    unpack8(ld_cached_v4(xr[r] + col), xf[r]);
#pragma unroll
                for (int j = 0; j < R; ++j) {
                    float wf[8];
                    unpack8(cur[j * Q + q], wf);
#pragma unroll
                    for (int r = 0; r < NR; ++r)
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            acc[j][r] = fmaf(wf[e], xf[r][e], acc[j][r]);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
            cur[i] = nxt[i];
    }
#pragma unroll
    for (int j = 0; j < R; ++j)
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
    rows_dot<4, NR>(w, H, xr, lane, acc);
    if (lane == 0) {
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            const float h0 = silu_f(acc[0][r]) * acc[2][r];
            const float h1 = silu_f(acc[1][r]) * acc[3][r];
            *reinterpret_cast<__nv_bfloat162 *>(hr[r] + i0) = __floats2bfloat162_rn(h0, h1);
        }
    }
}

// Down projection of LS_DOWN_ROWS output features f0, f0 + 1, ... over the columns [c0, c0 + ncols)
// of the intermediate for NR rows; partial sums to slot[f - f0][r] (shared memory).
template <int NR>
__device__ __forceinline__ void down_item(const __nv_bfloat16 *wd, int ld, int f0, int c0, int ncols,
                                          const __nv_bfloat16 *const (&hr)[NR], float *slot, int lane)
{
    const __nv_bfloat16 *w[LS_DOWN_ROWS];
#pragma unroll
    for (int j = 0; j < LS_DOWN_ROWS; ++j)
        w[j] = wd + (size_t)(f0 + j) * ld + c0;
    const __nv_bfloat16 *hc[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r)
        hc[r] = hr[r] + c0;
    float acc[LS_DOWN_ROWS][NR];
    rows_dot<LS_DOWN_ROWS, NR>(w, ncols, hc, lane, acc);
    if (lane == 0) {
#pragma unroll
        for (int j = 0; j < LS_DOWN_ROWS; ++j)
#pragma unroll
            for (int r = 0; r < NR; ++r)
                slot[j * LS_MAX_TOKENS + r] = acc[j][r];
    }
}

// ---- counters across the grid --------------------------------------------------------------------
//
// A 64-bit word: the call's epoch in the high half, a count in the low half.  The workspace need
// not be initialised and may hold the word of an earlier call (complete or abandoned): whoever
// finds another epoch there replaces the word by (epoch, own count); counts that went to the stale
// word meanwhile are repeated by their owners.
__device__ __forceinline__ void tagged_add(unsigned long long *word, uint32_t epoch)
{
    // count first: all but the call's first few arrivals find the epoch in place
    if ((uint32_t)(atomicAdd(word, 1ull) >> 32) == epoch)
        return;
    // the add went to a stale word: install (epoch, 1), or count again if somebody else has
    // installed the epoch meanwhile (adds to the stale word are dropped with it)
    const unsigned long long base = (unsigned long long)epoch << 32;
    unsigned long long seen = *reinterpret_cast<volatile unsigned long long *>(word);
    for (;;) {
        if ((uint32_t)(seen >> 32) == epoch) {
            atomicAdd(word, 1ull);
            return;
        }
        const unsigned long long prev = atomicCAS(word, seen, base + 1ull);
        if (prev == seen)
            return;
        seen = prev;
    }
}

// Bounded wait (one thread) until the word reads (epoch, target); acquire.  On giving up raises
// the status word and returns false.
__device__ __forceinline__ bool tagged_wait(const unsigned long long *word, uint32_t epoch,
                                            uint32_t target, int32_t *status, int wait_us)
{
    const unsigned long long want = ((unsigned long long)epoch << 32) + target;
    auto reached = [&]() {
        unsigned long long v;
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
        return v == want;
    };
    if (reached())
        return true;
    uint64_t t0;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i) {
            if (reached())
                return true;
            __nanosleep(40);
        }
        uint64_t t1;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
        if (t1 - t0 > 1000ull * (uint64_t)wait_us) {
            atomicExch(status, 1);
            return false;
        }
    }
}

// Named CTA barriers (id 1 .. 15; id 0 is __syncthreads): n threads in all arrive or wait.
__device__ __forceinline__ void named_sync(int id, int n)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory");
}
__device__ __forceinline__ void named_arrive(int id, int n)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory");
}

// Of the work items 0 .. n - 1, CTA b of G takes b, b + G, ...: how many that is.
__device__ __forceinline__ int owned_below(int n, int b, int G) { return n > b ? (n - b - 1) / G + 1 : 0; }

// Next index of a CTA-wide work queue (a counter in shared memory), the same in every lane.
__device__ __forceinline__ int pull(int *counter, int lane)
{
    int k = 0;
    if (lane == 0)
        k = atomicAdd(counter, 1);
    return __shfl_sync(0xffffffffu, k, 0);
}

// ---- the kernel -------------------------------------------------------------------------------

template <int VPL>
__global__ void __launch_bounds__(LS_THREADS, 1) layer_small_kernel(const SmallArgs a)
{
    extern __shared__ __align__(16) float s_slot[];        // partial sums of the CTA's down items
    __shared__ float s_z[LS_MAX_TOKENS][MOE_MAX_EXPERTS];  // logits of the call's tokens
    __shared__ float s_gate_w[LS_MAX_ASSIGN];              // by assignment t * K + j
    __shared__ int s_expert_of[LS_MAX_ASSIGN];             // by assignment
    __shared__ int s_group_of[LS_MAX_ASSIGN];              // by assignment: index of its expert's group
    __shared__ int s_row_of[LS_MAX_ASSIGN];                // by assignment: its row inside the group
    __shared__ int s_token_of[LS_MAX_ASSIGN];              // by sorted row
    __shared__ int s_leader[LS_MAX_ASSIGN];                // assignment is the first of its expert
    __shared__ int s_grp_expert[LS_MAX_ASSIGN], s_grp_row0[LS_MAX_ASSIGN], s_grp_n[LS_MAX_ASSIGN];
    __shared__ float s_shared_scale[LS_MAX_TOKENS];
    __shared__ int s_unit_left[LS_MAX_UNITS];  // gate/up items of the unit this CTA has yet to finish
    __shared__ int s_unit_ready[LS_MAX_UNITS];  // a warp of the CTA has seen the unit's gate/up complete
    __shared__ int s_q_shared, s_q_routed, s_q_down;  // work queues
    __shared__ int s_n_groups;
    __shared__ int s_ok;     // the grid barrier was passed
    __shared__ int s_abort;  // a wait gave up: leave

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, b = blockIdx.x;
    const int n_warps = G * LS_WARPS;
    const int gwarp = warp * G + b;  // consecutive work items land on different SMs
    const int T = a.T, H = a.H, E = a.E, K = a.K, A = a.T * a.K;
    const int n_shared_items = a.Is >> 1;  // gate/up items of the shared expert
    const int per_group = a.I >> 1;        // gate/up items of an activated expert

    if (tid == 0) {
        s_q_shared = s_q_routed = s_q_down = 0;
        s_abort = 0;
        s_ok = 0;
        s_unit_left[0] = owned_below(n_shared_items, b, G);
        for (int u = 0; u < LS_MAX_UNITS; ++u)
            s_unit_ready[u] = 0;
        if (b == 0)
            status_region_init(a.status);
    }
    __syncthreads();

    // Gate/up items of the shared expert, handed out to whichever warp asks.
    auto shared_gateup = [&]() {
        for (;;) {
            const int item = b + pull(&s_q_shared, lane) * G;
            if (item >= n_shared_items)
                break;
            const int i0 = item * 2;
#define LS_SHARED_GATEUP(NR)                                                             \
    {                                                                                    \
        const __nv_bfloat16 *xr[NR];                                                     \
        __nv_bfloat16 *hr[NR];                                                           \
        _Pragma("unroll") for (int r = 0; r < NR; ++r)                                   \
        {                                                                                \
            xr[r] = a.x + (size_t)r * H;                                                 \
            hr[r] = a.h_shared + (size_t)r * a.Is_pad;                                   \
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
            if (lane == 0) {
                __threadfence();  // h before the count
                if (atomicSub(&s_unit_left[0], 1) == 1) {
                    __threadfence();  // the other warps' h, seen through their counts
                    tagged_add(a.unit_done + 0, a.epoch);
                }
            }
        }
    };

    // ---- 1: partial logits ------------------------------------------------------------------------
    {
        const int rows = E + (a.gated ? 1 : 0);
        const int n_logit = rows * a.logit_chunks;
        for (int item = gwarp; item < n_logit; item += n_warps) {
            const int r = item / a.logit_chunks, c = item - r * a.logit_chunks;
            const int col0 = c * LS_LOGIT_CHUNK;
            constexpr int NQ = LS_LOGIT_CHUNK / 128;
            float acc[LS_MAX_TOKENS] = {0.f, 0.f, 0.f, 0.f};
            if (r < E) {
                const float *wr = a.w_router + (size_t)r * H;
                float4 wv[NQ];
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const int col = col0 + q * 128 + lane * 4;
                    wv[q] = col < H ? __ldg(reinterpret_cast<const float4 *>(wr + col))
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const int col = col0 + q * 128 + lane * 4;
                    if (col < H) {
#pragma unroll
                        for (int t = 0; t < LS_MAX_TOKENS; ++t) {
                            if (t < T) {
                                const uint2 xv = __ldg(
                                    reinterpret_cast<const uint2 *>(a.x + (size_t)t * H + col));
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
                for (int q = 0; q < NQ; ++q) {
                    const int col = col0 + q * 128 + lane * 4;
                    if (col < H) {
                        const uint2 wv = __ldg(reinterpret_cast<const uint2 *>(a.w_shared_gate + col));
#pragma unroll
                        for (int t = 0; t < LS_MAX_TOKENS; ++t) {
                            if (t < T) {
                                const uint2 xv = __ldg(
                                    reinterpret_cast<const uint2 *>(a.x + (size_t)t * H + col));
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
            if (lane == 0) {
                *reinterpret_cast<float4 *>(a.logit_part + (size_t)item * LS_MAX_TOKENS) =
                    make_float4(acc[0], acc[1], acc[2], acc[3]);
                __threadfence();
            }
        }
        __syncwarp();
    }

    // ---- 2: routing in four warps, the shared expert's gate/up in the others ------------------
    if (warp >= LS_ROUTE_WARPS) {
        named_arrive(1, LS_THREADS);  // this warp's partial logits are written
        shared_gateup();
        named_sync(3, LS_THREADS);  // the routing warps have filled the tables
    } else {
        constexpr int RT = LS_ROUTE_WARPS * 32;
        named_sync(1, LS_THREADS);  // every warp of the CTA has written its partial logits
        if (tid == 0) {
            __threadfence();
            tagged_add(a.barrier, a.epoch);
            s_ok = tagged_wait(a.barrier, a.epoch, G, a.status, a.wait_us) ? 1 : 0;
        }
        named_sync(2, RT);
        if (s_ok) {
            // logits = sum of the chunks in chunk order (+ bias); four (token, expert) pairs per
            // thread and pass, so that their loads are in flight together
            const int P = T * E;
            for (int idx0 = tid; idx0 < P; idx0 += 4 * RT) {
                float z[4] = {0.f, 0.f, 0.f, 0.f};
                const float *p[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int idx = min(idx0 + u * RT, P - 1);
                    const int t = idx / E, e = idx - t * E;
                    p[u] = a.logit_part + (size_t)e * a.logit_chunks * LS_MAX_TOKENS + t;
                }
                for (int c0 = 0; c0 < a.logit_chunks; c0 += 8) {
                    float v[8][4];
#pragma unroll
                    for (int c = 0; c < 8; ++c)
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            v[c][u] = c0 + c < a.logit_chunks ? __ldcg(p[u] + (c0 + c) * LS_MAX_TOKENS)
                                                              : 0.f;
#pragma unroll
                    for (int c = 0; c < 8; ++c)
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            z[u] += v[c][u];
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int idx = idx0 + u * RT;
                    if (idx < P) {
                        const int t = idx / E, e = idx - t * E;
                        const float v = z[u] + (a.router_bias != nullptr ? a.router_bias[e] : 0.f);
                        s_z[t][e] = v;
                        if (b == 0)
                            a.logits[idx] = v;
                    }
                }
            }
            if (a.gated && tid < T) {
                const float *p = a.logit_part + (size_t)E * a.logit_chunks * LS_MAX_TOKENS + tid;
                float z = 0.f;
                for (int c = 0; c < a.logit_chunks; ++c)
                    z += __ldcg(p + c * LS_MAX_TOKENS);
                const float sc = 1.0f / (1.0f + expf(-z));
                s_shared_scale[tid] = sc;
                if (b == 0)
                    a.shared_scale[tid] = sc;
            }
            named_sync(2, RT);
            if (warp < T) {
                const int t = warp;
                int sel_i;
                float sel_w;
                warp_route_topk<VPL>(s_z[t], E, K, a.score_fn, a.renormalize, a.routed_scale, lane,
                                     sel_i, sel_w);
                if (lane < K) {
                    s_expert_of[t * K + lane] = sel_i;
                    s_gate_w[t * K + lane] = sel_w;
                    if (b == 0) {
                        a.topk_idx[t * K + lane] = sel_i;
                        a.topk_w[t * K + lane] = sel_w;
                    }
                }
            }
            named_sync(2, RT);
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
                    s_group_of[lane] = groups_below;
                    s_row_of[lane] = rank;
                    s_token_of[pos] = lane / K;
                    if (leader) {
                        s_grp_expert[groups_below] = e;
                        s_grp_row0[groups_below] = less;
                        s_grp_n[groups_below] = __popc(peers);
                        // gate/up items of the group this CTA will finish
                        s_unit_left[1 + groups_below] =
                            owned_below((groups_below + 1) * per_group, b, G) -
                            owned_below(groups_below * per_group, b, G);
                    }
                    if (b == 0) {
                        a.perm[pos] = lane;
                        a.inv_perm[lane] = pos;
                    }
                }
                if (lane == 0)
                    s_n_groups = __popc(leaders);
            }
            named_sync(2, RT);
        }
        named_arrive(3, LS_THREADS);
        if (s_ok && b == 0) {
            // routing tables (copies for the caller; the kernel itself works from shared memory)
            for (int e = tid; e < E; e += RT) {
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
        if (s_ok)
            shared_gateup();  // whatever the other warps have left
    }
    if (!s_ok)
        return;  // every warp reads the flag behind barrier 2 or 3: all leave together

    // ---- 3: gate/up + SwiGLU of the activated experts, group by group -----------------------------
    {
        const int n_items = s_n_groups * per_group;
        for (;;) {
            const int item = b + pull(&s_q_routed, lane) * G;
            if (item >= n_items)
                break;
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
            hr[r] = a.h + (size_t)(row0 + r) * a.I_pad;                                  \
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
            if (lane == 0) {
                __threadfence();
                if (atomicSub(&s_unit_left[1 + g], 1) == 1) {
                    __threadfence();
                    tagged_add(a.unit_done + 1 + g, a.epoch);
                }
            }
        }
    }

    // ---- 4: down projection of the CTA's output features, unit by unit ------------------------
    const int n_blocks = H / LS_DOWN_ROWS;
    const int my_blocks = owned_below(n_blocks, b, G);
    const int n_uc = a.chunks_s + s_n_groups * a.chunks_r;  // (unit, column chunk) pairs
    {
        uint64_t ready = 0;  // units whose gate/up this warp has seen complete
        const int n_items = n_uc * my_blocks;
        for (;;) {
            if (*reinterpret_cast<volatile int *>(&s_abort))
                break;
            const int item = pull(&s_q_down, lane);
            if (item >= n_items)
                break;
            const int uc = item / my_blocks, k = item - uc * my_blocks;
            const int f0 = (b + k * G) * LS_DOWN_ROWS;
            int unit, c, n_done;
            if (uc < a.chunks_s) {
                unit = 0;
                c = uc;
                n_done = min(G, n_shared_items);
            } else {
                const int g = (uc - a.chunks_s) / a.chunks_r;
                unit = 1 + g;
                c = uc - a.chunks_s - g * a.chunks_r;
                n_done = min(G, per_group);
            }
            if (!((ready >> unit) & 1ull)) {
                // one acquire per CTA and unit: the first warp to need the unit waits for the
                // grid-wide counter and leaves a flag for the CTA's other warps
                int ok = 1;
                if (lane == 0) {
                    if (*reinterpret_cast<volatile int *>(&s_unit_ready[unit]) == 0) {
                        ok = tagged_wait(a.unit_done + unit, a.epoch, n_done, a.status, a.wait_us) ? 1 : 0;
                        __threadfence_block();
                        if (ok)
                            *reinterpret_cast<volatile int *>(&s_unit_ready[unit]) = 1;
                    } else {
                        __threadfence_block();
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) {
                    s_abort = 1;
                    break;
                }
                ready |= 1ull << unit;
            }
            float *slot = s_slot + (size_t)item * LS_SLOT_FLOATS;
            if (unit == 0) {
                const int c0 = c * a.chunk_s;
                const int ncols = min(a.chunk_s, a.Is - c0);
#define LS_SHARED_DOWN(NR)                                                               \
    {                                                                                    \
        const __nv_bfloat16 *hr[NR];                                                     \
        _Pragma("unroll") for (int r = 0; r < NR; ++r)                                   \
            hr[r] = a.h_shared + (size_t)r * a.Is_pad;                                   \
        down_item<NR>(a.ws_down, a.Is, f0, c0, ncols, hr, slot, lane);                   \
    }
                switch (T) {
                case 1: LS_SHARED_DOWN(1) break;
                case 2: LS_SHARED_DOWN(2) break;
                case 3: LS_SHARED_DOWN(3) break;
                default: LS_SHARED_DOWN(4) break;
                }
#undef LS_SHARED_DOWN
            } else {
                const int g = unit - 1;
                const int e = s_grp_expert[g], row0 = s_grp_row0[g], n = s_grp_n[g];
                const int c0 = c * a.chunk_r;
                const int ncols = min(a.chunk_r, a.I - c0);
                const __nv_bfloat16 *wd = a.w_down + (size_t)e * H * a.I;
#define LS_ROUTED_DOWN(NR)                                                               \
    {                                                                                    \
        const __nv_bfloat16 *hr[NR];                                                     \
        _Pragma("unroll") for (int r = 0; r < NR; ++r)                                   \
            hr[r] = a.h + (size_t)(row0 + r) * a.I_pad;                                  \
        down_item<NR>(wd, a.I, f0, c0, ncols, hr, slot, lane);                           \
    }
                switch (n) {
                case 1: LS_ROUTED_DOWN(1) break;
                case 2: LS_ROUTED_DOWN(2) break;
                case 3: LS_ROUTED_DOWN(3) break;
                default: LS_ROUTED_DOWN(4) break;
                }
#undef LS_ROUTED_DOWN
            }
        }
    }
    __syncthreads();
    if (s_abort)
        return;

    // ---- 5: combine the CTA's features -----------------------------------------------------------
    for (int idx = tid; idx < my_blocks * T; idx += LS_THREADS) {
        const int k = idx / T, t = idx - k * T;
        const int f0 = (b + k * G) * LS_DOWN_ROWS;
        float o[LS_DOWN_ROWS];
#pragma unroll
        for (int j = 0; j < LS_DOWN_ROWS; ++j)
            o[j] = 0.f;
        for (int slot_j = 0; slot_j < K; ++slot_j) {
            const int asg = t * K + slot_j;
            const int uc0 = a.chunks_s + s_group_of[asg] * a.chunks_r;
            const int r = s_row_of[asg];
            float y[LS_DOWN_ROWS];
#pragma unroll
            for (int j = 0; j < LS_DOWN_ROWS; ++j)
                y[j] = 0.f;
            for (int c = 0; c < a.chunks_r; ++c) {
                const float *slot = s_slot + ((size_t)(uc0 + c) * my_blocks + k) * LS_SLOT_FLOATS;
#pragma unroll
                for (int j = 0; j < LS_DOWN_ROWS; ++j)
                    y[j] += slot[j * LS_MAX_TOKENS + r];
            }
            const float gw = s_gate_w[asg];
#pragma unroll
            for (int j = 0; j < LS_DOWN_ROWS; ++j)
                o[j] = fmaf(gw, y[j], o[j]);
        }
        if (a.Is > 0) {
            float y[LS_DOWN_ROWS];
#pragma unroll
            for (int j = 0; j < LS_DOWN_ROWS; ++j)
                y[j] = 0.f;
            for (int c = 0; c < a.chunks_s; ++c) {
                const float *slot = s_slot + ((size_t)c * my_blocks + k) * LS_SLOT_FLOATS;
#pragma unroll
                for (int j = 0; j < LS_DOWN_ROWS; ++j)
                    y[j] += slot[j * LS_MAX_TOKENS + t];
            }
            const float sc = a.gated ? s_shared_scale[t] : 1.0f;
#pragma unroll
            for (int j = 0; j < LS_DOWN_ROWS; ++j)
                o[j] = fmaf(sc, y[j], o[j]);
        }
        static_assert(LS_DOWN_ROWS == 4, "the store below writes two bf16 pairs");
        const __nv_bfloat162 lo = __floats2bfloat162_rn(o[0], o[1]);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(o[2], o[3]);
        uint2 packed;
        packed.x = *reinterpret_cast<const uint32_t *>(&lo);
        packed.y = *reinterpret_cast<const uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(a.out + (size_t)t * H + f0) = packed;
    }
}

// ---- self-test of the bounded wait -------------------------------------------------------------

// Waits, with the given limit, for a counter that nothing advances: the wait of the one-launch
// layer (grid barrier, unit counters) must give up, raise the status word and return.  Word [3] of
// the status region records that it did.
__global__ void tagged_wait_selftest_kernel(int32_t *status, unsigned long long *never_reached,
                                            int limit_us)
{
    if (threadIdx.x == 0) {
        *never_reached = 0ull;
        status[3] = 0;
        __threadfence();
        const bool reached = tagged_wait(never_reached, 0xffffffffu, 1u, status, limit_us);
        status[3] = reached ? 0 : 1;
    }
}

cudaError_t launch_tagged_wait_selftest(int32_t *status, int limit_us, cudaStream_t s)
{
    tagged_wait_selftest_kernel<<<1, 32, 0, s>>>(
        status, reinterpret_cast<unsigned long long *>(status + LS_SELFTEST_WORD), limit_us);
    return cudaGetLastError();
}

// ---- host -------------------------------------------------------------------------------------

// Most columns of a down-projection item for this shape: long items stream best, but a CTA needs
// a few items per warp to keep all of them busy -- the longest chunk that leaves it
// LS_DOWN_ITEMS_WANTED items at one token (T = 1: top_k groups), else the shortest.
static int down_chunk_limit(const moe_config_t &c)
{
    const int blocks = (c.hidden / LS_DOWN_ROWS + sm_count() - 1) / sm_count();
    for (int chunk = LS_DOWN_CHUNK_MAX; chunk > LS_DOWN_CHUNK_MIN; chunk /= 2) {
        const int uc = (c.shared_inter + chunk - 1) / chunk + c.top_k * ((c.inter + chunk - 1) / chunk);
        if (uc * blocks >= LS_DOWN_ITEMS_WANTED)
            return chunk;
    }
    return LS_DOWN_CHUNK_MIN;
}

static int down_chunks(const moe_config_t &c, int cols)
{
    const int limit = down_chunk_limit(c);
    return (cols + limit - 1) / limit;
}

// columns per chunk: equal shares, rounded up to whole parts of the row walk
static int down_chunk_cols(const moe_config_t &c, int cols)
{
    const int n = down_chunks(c, cols);
    return n == 0 ? 0 : (((cols + n - 1) / n) + 255) & ~255;
}

static size_t pitch(int cols) { return ((size_t)cols + 63) & ~(size_t)63; }  // elements: 128-byte lines

// shared memory for the partial sums of one CTA's down-projection items
static size_t slot_bytes(const moe_config_t &c, int T)
{
    const size_t blocks = ((size_t)c.hidden / LS_DOWN_ROWS + sm_count() - 1) / sm_count();
    const size_t uc = (size_t)down_chunks(c, c.shared_inter) + (size_t)T * c.top_k * down_chunks(c, c.inter);
    return uc * blocks * LS_SLOT_FLOATS * sizeof(float);
}

static bool small_shape(const moe_config_t &c, int T)
{
    if (T > LS_MAX_TOKENS || T * c.top_k > LS_MAX_ASSIGN || slot_bytes(c, T) > LS_MAX_SLOT_BYTES)
        return false;
    // The shared expert multiplies every weight with all T rows on the CUDA cores; with a large
    // shared expert and more than one row that falls behind the weight stream, and the kernel
    // chain (tensor cores) is the faster path (measured crossover).
    return T == 1 || (size_t)T * c.shared_inter * c.hidden <= LS_SHARED_WORK_MAX;
}

// the largest T' <= T the one-launch kernel takes (0: none)
static int largest_small(const moe_config_t &c, int T)
{
    int t = T < LS_MAX_TOKENS ? T : LS_MAX_TOKENS;
    while (t > 0 && !small_shape(c, t))
        --t;
    return t;
}

size_t layer_small_logit_part_bytes(const moe_config_t &c)
{
    const size_t chunks = (c.hidden + LS_LOGIT_CHUNK - 1) / LS_LOGIT_CHUNK;
    return LS_UNIT_WORD_BYTES + ((size_t)c.n_experts + 1) * chunks * LS_MAX_TOKENS * sizeof(float);
}

// sized for the largest small call, so that the layout never shrinks as T grows
size_t layer_small_h_bytes(const moe_config_t &c, int T)
{
    const int t = largest_small(c, T);
    return ((size_t)t * c.top_k * pitch(c.inter) + (size_t)t * pitch(c.shared_inter)) * 2;
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

template <int VPL>
static cudaError_t launch_variant(const SmallArgs &a, size_t smem, cudaStream_t s)
{
    static DeviceOnce configured;
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess)
        return err;
    if (!configured.done(dev)) {
        err = cudaFuncSetAttribute(layer_small_kernel<VPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)LS_MAX_SLOT_BYTES);
        if (err != cudaSuccess)
            return err;
        configured.mark(dev);
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(sm_count());
    cfg.blockDim = dim3(LS_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, layer_small_kernel<VPL>, a);
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
    a.unit_done = reinterpret_cast<unsigned long long *>(ws + L.small_logit_part);
    a.logit_part = reinterpret_cast<float *>(ws + L.small_logit_part + LS_UNIT_WORD_BYTES);
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
    a.I_pad = (int)pitch(c.inter);
    a.Is_pad = (int)pitch(c.shared_inter);
    a.h = reinterpret_cast<__nv_bfloat16 *>(ws + L.small_h);
    a.h_shared = a.h + (size_t)T * c.top_k * a.I_pad;
    a.status = reinterpret_cast<int32_t *>(ws + L.status);
    a.barrier = reinterpret_cast<unsigned long long *>(a.status + LS_BARRIER_WORD);
    a.epoch = epoch;
    a.wait_us = (int)(LS_WAIT_NS / 1000ull);
    a.logit_chunks = (c.hidden + LS_LOGIT_CHUNK - 1) / LS_LOGIT_CHUNK;
    a.chunks_r = down_chunks(c, c.inter);
    a.chunk_r = down_chunk_cols(c, c.inter);
    a.chunks_s = down_chunks(c, c.shared_inter);
    a.chunk_s = down_chunk_cols(c, c.shared_inter);
    const size_t smem = slot_bytes(c, T);
    const int E = c.n_experts;
    if (E <= 32)
        return launch_variant<1>(a, smem, s);
    if (E <= 64)
        return launch_variant<2>(a, smem, s);
    if (E <= 128)
        return launch_variant<4>(a, smem, s);
    if (E <= 256)
        return launch_variant<8>(a, smem, s);
    return launch_variant<16>(a, smem, s);
}

}  // namespace moe

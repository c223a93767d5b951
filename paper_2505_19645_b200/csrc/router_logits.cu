// Router logits  z[t,e] = x[t,:] . w_router[e,:] (+ bias[e])  and the shared expert's scalar
// gate  s[t] = sigmoid(x[t,:] . w_sg), with fp32-level accuracy on the tensor cores.
//
// The fp32 router row is split on the fly into three bf16 terms  w = hi + mid + lo  (each
// remainder is exact in fp32, so the three terms carry 24 mantissa bits), the bf16 token
// values are exact, and the three partial products are accumulated in fp32 by
// m16n8k16 MMAs.  A CTA owns 16 router rows x (8*NCH) tokens; its 16 warps split H and are
// summed through shared memory, so even T = 1 keeps every load short and parallel.
#include <cooperative_groups.h>

#include "common.cuh"

namespace moe {

namespace cg = cooperative_groups;

// warps per CTA (they split H): 16 for the small token tiles that latency-bound calls use
#define RL_WARPS_FOR(nch) ((nch) <= 2 ? 16 : 8)

struct Split3 {
    uint32_t hi, mid, lo;  // two bf16 each
};

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b)
{
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&p);
}

__device__ __forceinline__ Split3 split_pair(float a, float b)
{
    Split3 s;
    s.hi = pack_bf16x2(a, b);
    const float ra = a - bf16_lo(s.hi), rb = b - bf16_hi(s.hi);
    s.mid = pack_bf16x2(ra, rb);
    const float ra2 = ra - bf16_lo(s.mid), rb2 = rb - bf16_hi(s.mid);
    s.lo = pack_bf16x2(ra2, rb2);
    return s;
}

// 8 consecutive values of one router row as fp32 (row kinds: fp32 router row, the bf16
// shared-gate vector, or a padding row of zeros).
struct RowSrc {
    const float *f32;           // non-null: fp32 row
    const __nv_bfloat16 *bf16;  // non-null: bf16 row
};

__device__ __forceinline__ void load_row8(const RowSrc &r, int k, float (&v)[8])
{
    if (r.f32) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(r.f32 + k));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(r.f32 + k + 4));
        v[0] = a.x, v[1] = a.y, v[2] = a.z, v[3] = a.w;
        v[4] = b.x, v[5] = b.y, v[6] = b.z, v[7] = b.w;
    } else if (r.bf16) {
        const uint4 p = __ldg(reinterpret_cast<const uint4 *>(r.bf16 + k));
        v[0] = bf16_lo(p.x), v[1] = bf16_hi(p.x), v[2] = bf16_lo(p.y), v[3] = bf16_hi(p.y);
        v[4] = bf16_lo(p.z), v[5] = bf16_hi(p.z), v[6] = bf16_lo(p.w), v[7] = bf16_hi(p.w);
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            v[i] = 0.f;
    }
}

// Sum of the warps' partial accumulators of one block of 16 router rows, written out.
template <int NCH>
__device__ __forceinline__ void reduce_and_store(const float (&part)[RL_WARPS_FOR(NCH)][NCH][4][32],
                                                 int e0, int t0, int T, int E, int n_rows,
                                                 const float *__restrict__ bias,
                                                 float *__restrict__ logits,
                                                 float *__restrict__ shared_scale)
{
    constexpr int RL_WARPS = RL_WARPS_FOR(NCH);
    // accumulator q of lane (g,tq), chunk c: row g + 8*(q>>1), token c*8 + 2*tq + (q&1)
    for (int o = threadIdx.x; o < 16 * 8 * NCH; o += RL_WARPS * 32) {
        const int r = o & 15, slot = o >> 4;
        const int c = slot >> 3, tt = (slot & 7) >> 1, lo = slot & 1;
        const int q = ((r >> 3) << 1) | lo, ln = ((r & 7) << 2) | tt;
        const int e = e0 + r, t = t0 + slot;
        if (e >= n_rows || t >= T)
            continue;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < RL_WARPS; ++w)
            v += part[w][c][q][ln];
        if (e < E)
            logits[(size_t)t * E + e] = bias ? v + bias[e] : v;
        else
            shared_scale[t] = 1.0f / (1.0f + expf(-v));
    }
}

// The same for a cluster of CTAs that split H between them (few tokens, few row blocks: one CTA
// per row block would leave most SMs idle and each CTA a long reduction).  Every CTA sums its
// warps into `red`; the cluster's first CTA adds the CTAs' sums in rank order through
// distributed shared memory -- a fixed order, so the logits do not depend on timing.
template <int NCH>
__device__ __forceinline__ void reduce_cluster_and_store(
    const float (&part)[RL_WARPS_FOR(NCH)][NCH][4][32], float (&red)[16 * 8 * NCH], int e0, int t0,
    int T, int E, int n_rows, const float *__restrict__ bias, float *__restrict__ logits,
    float *__restrict__ shared_scale)
{
    constexpr int RL_WARPS = RL_WARPS_FOR(NCH);
    cg::cluster_group cluster = cg::this_cluster();
    for (int o = threadIdx.x; o < 16 * 8 * NCH; o += RL_WARPS * 32) {
        const int r = o & 15, slot = o >> 4;
        const int c = slot >> 3, tt = (slot & 7) >> 1, lo = slot & 1;
        const int q = ((r >> 3) << 1) | lo, ln = ((r & 7) << 2) | tt;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < RL_WARPS; ++w)
            v += part[w][c][q][ln];
        red[o] = v;
    }
    cluster.sync();
    if (cluster.block_rank() == 0) {
        const unsigned n = cluster.num_blocks();
        for (int o = threadIdx.x; o < 16 * 8 * NCH; o += RL_WARPS * 32) {
            const int r = o & 15, slot = o >> 4;
            const int e = e0 + r, t = t0 + slot;
            if (e >= n_rows || t >= T)
                continue;
            float v = red[o];
            for (unsigned k = 1; k < n; ++k)
                v += cluster.map_shared_rank(&red[0], k)[o];
            if (e < E)
                logits[(size_t)t * E + e] = bias ? v + bias[e] : v;
            else
                shared_scale[t] = 1.0f / (1.0f + expf(-v));
        }
    }
    cluster.sync();  // the other CTAs' shared memory stays valid until it has been read
}

// RB: blocks of 16 router rows per CTA.  With many experts and many tokens the kernel is bound by
// what its CTAs re-read from L2 (every token tile once per row block, every row block once per
// token tile); two row blocks per CTA share the token loads and halve the first term.
template <int NCH, int RB>
__global__ void __launch_bounds__(RL_WARPS_FOR(NCH) * 32)
router_logits_kernel(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ w_router,
                     const float *__restrict__ bias, const __nv_bfloat16 *__restrict__ w_sg,
                     int T, int H, int E, int n_rows, float *__restrict__ logits,
                     float *__restrict__ shared_scale, int32_t *__restrict__ zero, int zero_n,
                     int32_t *__restrict__ status)
{
    constexpr int RL_WARPS = RL_WARPS_FOR(NCH);
    __shared__ float part[RL_WARPS][NCH][4][32];
    griddep_wait();    // first kernel of a layer call: everything older is complete from here on
    if ((zero != nullptr || status != nullptr) && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) {
        // counters that a later kernel of this call updates before the plan kernel has run
        for (int i = threadIdx.x; i < zero_n; i += blockDim.x)
            zero[i] = 0;
        if (threadIdx.x == 0)
            status_region_init(status);
        __threadfence();
        __syncthreads();
    }
    griddep_launch();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int e0 = blockIdx.x * 16 * RB;
    const int t0 = blockIdx.y * (8 * NCH);

    auto row_src = [&](int e) {
        RowSrc r{nullptr, nullptr};
        if (e < E)
            r.f32 = w_router + (size_t)e * H + 8 * tq;
        else if (e == E && e < n_rows)
            r.bf16 = w_sg + 8 * tq;
        return r;
    };
    RowSrc rlo[RB], rhi[RB];
#pragma unroll
    for (int rb = 0; rb < RB; ++rb) {
        rlo[rb] = row_src(e0 + 16 * rb + g);
        rhi[rb] = row_src(e0 + 16 * rb + g + 8);
    }
    const __nv_bfloat16 *b[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c)
        b[c] = x + (size_t)min(t0 + c * 8 + g, T - 1) * H + 8 * tq;

    float acc[RB][NCH][4];
#pragma unroll
    for (int rb = 0; rb < RB; ++rb)
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
            for (int q = 0; q < 4; ++q)
                acc[rb][c][q] = 0.f;

    // gridDim.z CTAs (one cluster) split H; the warps of a CTA split the CTA's share
    const int nsteps_all = H >> 5;
    const int z0 = blockIdx.z * nsteps_all / gridDim.z, z1 = (blockIdx.z + 1) * nsteps_all / gridDim.z;
    const int nsteps = z1 - z0;
    const int s0 = z0 + warp * nsteps / RL_WARPS, s1 = z0 + (warp + 1) * nsteps / RL_WARPS;
#pragma unroll 4
    for (int s = s0; s < s1; ++s) {
        const int k = s * 32;
        uint4 B[NCH];
#pragma unroll
        for (int c = 0; c < NCH; ++c)
            B[c] = ld_cached_v4(b[c] + k);
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) {
            float lo8[8], hi8[8];
            load_row8(rlo[rb], k, lo8);
            load_row8(rhi[rb], k, hi8);
            // physical k positions 8tq+{0..3} feed the first MMA, 8tq+{4..7} the second
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const Split3 a0 = split_pair(lo8[4 * half + 0], lo8[4 * half + 1]);
                const Split3 a1 = split_pair(hi8[4 * half + 0], hi8[4 * half + 1]);
                const Split3 a2 = split_pair(lo8[4 * half + 2], lo8[4 * half + 3]);
                const Split3 a3 = split_pair(hi8[4 * half + 2], hi8[4 * half + 3]);
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    const uint32_t b0 = half ? B[c].z : B[c].x, b1 = half ? B[c].w : B[c].y;
                    mma_bf16_16816(acc[rb][c], a0.lo, a1.lo, a2.lo, a3.lo, b0, b1);
                    mma_bf16_16816(acc[rb][c], a0.mid, a1.mid, a2.mid, a3.mid, b0, b1);
                    mma_bf16_16816(acc[rb][c], a0.hi, a1.hi, a2.hi, a3.hi, b0, b1);
                }
            }
        }
    }

#pragma unroll
    for (int rb = 0; rb < RB; ++rb) {
        if (rb > 0)
            __syncthreads();  // the previous row block's sums have been read
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
            for (int q = 0; q < 4; ++q)
                part[warp][c][q][lane] = acc[rb][c][q];
        __syncthreads();
        if constexpr (RB == 1 && NCH == 1) {
            if (gridDim.z > 1) {
                __shared__ float red[16 * 8 * NCH];
                reduce_cluster_and_store<NCH>(part, red, e0, t0, T, E, n_rows, bias, logits,
                                              shared_scale);
                continue;
            }
        }
        reduce_and_store<NCH>(part, e0 + 16 * rb, t0, T, E, n_rows, bias, logits, shared_scale);
    }
}

cudaError_t launch_router_logits(const moe_config_t &c, const moe_weights_t &w,
                                 const __nv_bfloat16 *x, int T, float *logits,
                                 float *shared_scale, cudaStream_t s, int32_t *zero, int zero_n,
                                 int32_t *status)
{
    const bool gate_row = shared_scale != nullptr && c.shared_gate && c.shared_inter > 0;
    const int n_rows = c.n_experts + (gate_row ? 1 : 0);
    const int e_tiles = (n_rows + 15) / 16;
    // the smallest token tile that keeps the grid within one wave (a CTA of 16 warps fills an SM)
    int nch = 1;
    while (nch < 8 && (long long)e_tiles * ((T + 8 * nch - 1) / (8 * nch)) > (long long)sm_count())
        nch *= 2;
    // two row blocks per CTA once the grid exceeds a wave of the largest token tile
    const int token_tiles = (T + 8 * nch - 1) / (8 * nch);
    const int rb = (nch == 8 && e_tiles >= 8 && (long long)e_tiles * token_tiles > (long long)sm_count()) ? 2 : 1;
    dim3 grid((e_tiles + rb - 1) / rb, token_tiles);
    // Few row blocks and few tokens with a long reduction (eight and more 32-element steps per
    // warp: below that the cluster launch costs what the shorter loops save): clusters of up
    // to eight CTAs split H, as long as the grid stays within one wave and every warp keeps at
    // least one step.
    int ks = 1;
    if (nch == 1 && (c.hidden >> 5) / RL_WARPS_FOR(1) >= 8) {
        ks = 8;
        while (ks > 1 && ((long long)e_tiles * token_tiles * ks > (long long)sm_count() ||
                          (c.hidden >> 5) / ks < RL_WARPS_FOR(1)))
            ks /= 2;
    }
    if (ks > 1) {
        grid.z = ks;
        void (*kernel)(const __nv_bfloat16 *, const float *, const float *, const __nv_bfloat16 *, int,
                       int, int, int, float *, float *, int32_t *, int, int32_t *) = router_logits_kernel<1, 1>;
        prefer_max_shared_carveout(reinterpret_cast<const void *>(kernel));
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(RL_WARPS_FOR(1) * 32);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = s;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 1;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = ks;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        return cudaLaunchKernelEx(&cfg, kernel, x, w.w_router, w.router_bias,
                                  static_cast<const __nv_bfloat16 *>(w.w_shared_gate), T, c.hidden,
                                  c.n_experts, n_rows, logits, shared_scale, zero, zero_n, status);
    }
    const __nv_bfloat16 *w_sg = static_cast<const __nv_bfloat16 *>(w.w_shared_gate);
#define MOE_RL_LAUNCH(N, R)                                                                 \
    err = launch_pdl(router_logits_kernel<N, R>, grid, dim3(RL_WARPS_FOR(N) * 32), 0, s, x, w.w_router, \
                     w.router_bias, w_sg, T, c.hidden, c.n_experts, n_rows, logits, shared_scale, zero,  \
                     zero_n, status)
    cudaError_t err = cudaSuccess;
    switch (nch) {
    case 1: MOE_RL_LAUNCH(1, 1); break;
    case 2: MOE_RL_LAUNCH(2, 1); break;
    case 4: MOE_RL_LAUNCH(4, 1); break;
    default:
        if (rb == 2)
            MOE_RL_LAUNCH(8, 2);
        else
            MOE_RL_LAUNCH(8, 1);
        break;
    }
#undef MOE_RL_LAUNCH
    return err;
}

}  // namespace moe

// Router: fp32 logits (x . w_router^T + bias), the shared expert's scalar gate, and the
// warp-per-token top-k selection with softmax / sigmoid gate weights.
#include <float.h>

#include "common.cuh"

namespace moe {

// ---------------------------------------------------------------------------------------
// Router logits.  One warp owns one router row (expert) and a block of TOK tokens; lanes
// stride over H with 128-bit loads of the fp32 row and 64-bit loads of the bf16 tokens.
// The 8 warps of a CTA share the token block, so the token rows hit in L1.
// Virtual row E (when present) is the bf16 shared-gate vector; its result goes through a
// sigmoid into shared_scale.
// ---------------------------------------------------------------------------------------
constexpr int RL_TOK = 8;
constexpr int RL_WARPS = 8;

__global__ void __launch_bounds__(RL_WARPS * 32)
router_logits_kernel(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ w_router,
                     const float *__restrict__ bias, const __nv_bfloat16 *__restrict__ w_sg,
                     int T, int H, int E, int n_rows, float *__restrict__ logits,
                     float *__restrict__ shared_scale)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int e = blockIdx.x * RL_WARPS + warp;
    const int t0 = blockIdx.y * RL_TOK;
    if (e >= n_rows)
        return;
    const bool is_gate_row = (e == E);
    float acc[RL_TOK];
#pragma unroll
    for (int i = 0; i < RL_TOK; ++i)
        acc[i] = 0.f;
    const __nv_bfloat16 *xr[RL_TOK];
#pragma unroll
    for (int i = 0; i < RL_TOK; ++i)
        xr[i] = x + (size_t)min(t0 + i, T - 1) * H;

    for (int h = lane * 4; h < H; h += 128) {
        float4 wv;
        if (!is_gate_row) {
            wv = __ldg(reinterpret_cast<const float4 *>(w_router + (size_t)e * H + h));
        } else {
            const uint2 p = __ldg(reinterpret_cast<const uint2 *>(w_sg + h));
            wv = make_float4(bf16_lo(p.x), bf16_hi(p.x), bf16_lo(p.y), bf16_hi(p.y));
        }
#pragma unroll
        for (int i = 0; i < RL_TOK; ++i) {
            const uint2 p = *reinterpret_cast<const uint2 *>(xr[i] + h);
            acc[i] = fmaf(bf16_lo(p.x), wv.x, acc[i]);
            acc[i] = fmaf(bf16_hi(p.x), wv.y, acc[i]);
            acc[i] = fmaf(bf16_lo(p.y), wv.z, acc[i]);
            acc[i] = fmaf(bf16_hi(p.y), wv.w, acc[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < RL_TOK; ++i) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1)
            acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], off);
    }
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < RL_TOK; ++i) {
            const int t = t0 + i;
            if (t >= T)
                break;
            if (!is_gate_row) {
                float z = acc[i];
                if (bias)
                    z += bias[e];
                logits[(size_t)t * E + e] = z;
            } else {
                shared_scale[t] = 1.0f / (1.0f + expf(-acc[i]));
            }
        }
    }
}

cudaError_t launch_router_logits(const moe_config_t &c, const moe_weights_t &w,
                                 const __nv_bfloat16 *x, int T, float *logits,
                                 float *shared_scale, cudaStream_t s)
{
    const bool gate_row = shared_scale != nullptr && c.shared_gate && c.shared_inter > 0;
    const int n_rows = c.n_experts + (gate_row ? 1 : 0);
    dim3 grid((n_rows + RL_WARPS - 1) / RL_WARPS, (T + RL_TOK - 1) / RL_TOK);
    router_logits_kernel<<<grid, RL_WARPS * 32, 0, s>>>(
        x, w.w_router, w.router_bias, static_cast<const __nv_bfloat16 *>(w.w_shared_gate), T,
        c.hidden, c.n_experts, n_rows, logits, shared_scale);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Top-k.  One warp per token; lane l holds logits l, l+32, ...  Selection runs k rounds of
// a warp arg-max on the raw fp32 logits (ties: lower expert index), so it is exact and
// independent of the score function.  Scores use expf.
// ---------------------------------------------------------------------------------------
template <int VPL>
__global__ void __launch_bounds__(128)
route_topk_kernel(const float *__restrict__ logits, int T, int E, int k, int score_fn,
                  int renormalize, float routed_scale, int32_t *__restrict__ topk_idx,
                  float *__restrict__ topk_w)
{
    const int lane = threadIdx.x & 31;
    const int t = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5);
    if (t >= T)
        return;
    const float *z = logits + (size_t)t * E;
    float v[VPL];
    float vmax = -FLT_MAX;
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
        const int e = lane + 32 * i;
        v[i] = e < E ? z[e] : -FLT_MAX;
        vmax = fmaxf(vmax, v[i]);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, off));
    float denom = 1.f;
    if (score_fn == MOE_SCORE_SOFTMAX) {
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < VPL; ++i)
            if (lane + 32 * i < E)
                sum += expf(v[i] - vmax);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1)
            sum += __shfl_xor_sync(0xffffffffu, sum, off);
        denom = sum;
    }

    uint32_t taken = 0;
    float sel_v = 0.f;
    int sel_i = 0;
    for (int j = 0; j < k; ++j) {
        float bv = -FLT_MAX;
        int bi = 0x7fffffff;
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
            const int e = lane + 32 * i;
            if (e < E && !((taken >> i) & 1u) && (bi == 0x7fffffff || v[i] > bv)) {
                bv = v[i];
                bi = e;
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            if (oi != 0x7fffffff && (bi == 0x7fffffff || ov > bv || (ov == bv && oi < bi))) {
                bv = ov;
                bi = oi;
            }
        }
        if (bi != 0x7fffffff && (bi & 31) == lane)
            taken |= 1u << (bi >> 5);
        if (lane == j) {
            sel_v = bv;
            sel_i = bi;
        }
    }
    float p = 0.f;
    if (lane < k) {
        if (score_fn == MOE_SCORE_SOFTMAX)
            p = expf(sel_v - vmax) / denom;
        else
            p = 1.0f / (1.0f + expf(-sel_v));
    }
    if (renormalize) {
        float s = p;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1)
            s += __shfl_xor_sync(0xffffffffu, s, off);
        p = p / s;
    }
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = sel_i;
        topk_w[(size_t)t * k + lane] = p * routed_scale;
    }
}

cudaError_t launch_route_topk(const moe_config_t &c, const float *logits, int T, int32_t *idx,
                              float *wts, cudaStream_t s)
{
    const int E = c.n_experts;
    const int threads = 128;
    const int blocks = (int)(((size_t)T * 32 + threads - 1) / threads);
#define MOE_TOPK_LAUNCH(V)                                                                     \
    route_topk_kernel<V><<<blocks, threads, 0, s>>>(logits, T, E, c.top_k, c.score_fn,        \
                                                   c.renormalize, c.routed_scale, idx, wts)
    if (E <= 32)
        MOE_TOPK_LAUNCH(1);
    else if (E <= 64)
        MOE_TOPK_LAUNCH(2);
    else if (E <= 128)
        MOE_TOPK_LAUNCH(4);
    else if (E <= 256)
        MOE_TOPK_LAUNCH(8);
    else
        MOE_TOPK_LAUNCH(16);
#undef MOE_TOPK_LAUNCH
    return cudaGetLastError();
}

}  // namespace moe

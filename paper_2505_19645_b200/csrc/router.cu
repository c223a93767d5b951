// Router: fp32 logits (x . w_router^T + bias), the shared expert's scalar gate, and the
// warp-per-token top-k selection with softmax / sigmoid gate weights.
#include <float.h>

#include "common.cuh"

namespace moe {


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
    griddep_launch();
    griddep_wait();  // the logits come from the preceding kernel
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
    err = launch_pdl(route_topk_kernel<V>, dim3(blocks), dim3(threads), 0, s, logits, T, E,    \
                     c.top_k, c.score_fn, c.renormalize, c.routed_scale, idx, wts)
    cudaError_t err = cudaSuccess;
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
    return err;
}

}  // namespace moe

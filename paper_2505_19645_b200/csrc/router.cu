// Top-k routing kernel: one warp per token selects the k experts and their softmax / sigmoid
// gate weights from the fp32 logits.
#include "route_topk.cuh"

namespace moe {

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
    int sel_i;
    float sel_w;
    warp_route_topk<VPL>(logits + (size_t)t * E, E, k, score_fn, renormalize, routed_scale, lane,
                         sel_i, sel_w);
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = sel_i;
        topk_w[(size_t)t * k + lane] = sel_w;
    }
}

// The same for large batches whose logits arrive as partial sums per k chunk (tensor-core logit
// path): the warp first adds its token's chunks in chunk order -- lane l the experts l, l + 32, ...
// it will rank anyway --, stores the logits, then selects from what it stored.
template <int VPL>
__global__ void __launch_bounds__(128)
route_topk_sum_kernel(const float *__restrict__ partial, int chunks, int R,
                      const float *__restrict__ bias, int T, int E, int k, int score_fn,
                      int renormalize, float routed_scale, float *__restrict__ logits,
                      float *__restrict__ shared_scale, int32_t *__restrict__ topk_idx,
                      float *__restrict__ topk_w)
{
    griddep_launch();
    griddep_wait();  // the partial sums come from the preceding kernel
    const int lane = threadIdx.x & 31;
    const int t = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5);
    if (t >= T)
        return;
    const size_t plane = (size_t)T * R;
    const float *p = partial + (size_t)t * R;
    float v[VPL];
#pragma unroll
    for (int i = 0; i < VPL; ++i)
        v[i] = 0.f;
    for (int s = 0; s < chunks; ++s) {
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
            const int e = lane + 32 * i;
            if (e < E)
                v[i] += __ldg(p + (size_t)s * plane + e);
        }
    }
    float *z = logits + (size_t)t * E;
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
        const int e = lane + 32 * i;
        if (e < E)
            z[e] = bias != nullptr ? v[i] + bias[e] : v[i];
    }
    if (shared_scale != nullptr && lane == 0) {
        float g = 0.f;
        for (int s = 0; s < chunks; ++s)
            g += __ldg(p + (size_t)s * plane + E);
        shared_scale[t] = 1.0f / (1.0f + expf(-g));
    }
    __syncwarp();  // (every lane re-reads only what it stored itself)
    int sel_i;
    float sel_w;
    warp_route_topk<VPL>(z, E, k, score_fn, renormalize, routed_scale, lane, sel_i, sel_w);
    if (lane < k) {
        topk_idx[(size_t)t * k + lane] = sel_i;
        topk_w[(size_t)t * k + lane] = sel_w;
    }
}

cudaError_t launch_route_topk_sum(const moe_config_t &c, const float *partial, int chunks, int R,
                                  const float *bias, int T, float *logits, float *shared_scale,
                                  int32_t *idx, float *wts, cudaStream_t s)
{
    const int E = c.n_experts;
    const int threads = 128;
    const int blocks = (int)(((size_t)T * 32 + threads - 1) / threads);
#define MOE_TOPK_SUM_LAUNCH(V)                                                                  \
    err = launch_pdl(route_topk_sum_kernel<V>, dim3(blocks), dim3(threads), 0, s, partial,      \
                     chunks, R, bias, T, E, c.top_k, c.score_fn, c.renormalize, c.routed_scale, \
                     logits, shared_scale, idx, wts)
    cudaError_t err = cudaSuccess;
    if (E <= 32)
        MOE_TOPK_SUM_LAUNCH(1);
    else if (E <= 64)
        MOE_TOPK_SUM_LAUNCH(2);
    else if (E <= 128)
        MOE_TOPK_SUM_LAUNCH(4);
    else if (E <= 256)
        MOE_TOPK_SUM_LAUNCH(8);
    else
        MOE_TOPK_SUM_LAUNCH(16);
#undef MOE_TOPK_SUM_LAUNCH
    return err;
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

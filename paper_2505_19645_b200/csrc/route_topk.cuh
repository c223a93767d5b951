// Top-k selection and gate weights of one token by one warp (Sec. 3.2: each token activates
// K of the E experts).  Lane l holds logits l, l+32, ...; selection runs k rounds of a warp
// arg-max on the raw fp32 logits (ties: lower expert index), so it is exact and independent
// of the score function.  Scores use expf.
#pragma once
#include <float.h>

#include "common.cuh"

namespace moe {

// All 32 lanes call it with the token's logits z[0..E).  On return lane j < k holds the j-th
// selected expert in sel_i and its gate weight (already multiplied by routed_scale) in sel_w.
template <int VPL>
__device__ __forceinline__ void warp_route_topk(const float *__restrict__ z, int E, int k,
                                                int score_fn, int renormalize, float routed_scale,
                                                int lane, int &sel_i, float &sel_w)
{
    float v[VPL];
    float vmax = -FLT_MAX;
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
        const int e = lane + 32 * i;
        v[i] = e < E ? z[e] : -FLT_MAX;
        if (!(v[i] == v[i]))
            v[i] = -FLT_MAX;  // NaN (outside the contract) ranks lowest: the arg-max below needs
                              // a total order for all lanes to agree, else an index could be lost
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
    sel_i = 0;
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
    sel_w = p * routed_scale;
}

}  // namespace moe

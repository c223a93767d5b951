// Gate-weighted combine: out[t] = sum_j w[t,j] * y[inv_perm[t*K+j]] + s[t] * shared_y[t]
// (y and shared_y may arrive as partial planes, one per k chunk of the down projection).
// Gather form (each output row is summed in slot order by one owner), so the result does
// not depend on scheduling; 128-bit loads and stores.
#include "common.cuh"

namespace moe {

constexpr int CB_THREADS = 256;
constexpr int MOE_MAX_SHARED_PARTS = 8;  // k chunks of the shared expert's down pass, at most

__global__ void __launch_bounds__(CB_THREADS)
combine_kernel(const __nv_bfloat16 *__restrict__ y, int routed_parts,
               const int32_t *__restrict__ inv_perm,
               const float *__restrict__ topk_w, const __nv_bfloat16 *__restrict__ shared_y,
               int shared_parts, const float *__restrict__ shared_scale, int T, int H, int k,
               __nv_bfloat16 *__restrict__ out)
{
    griddep_launch();
    griddep_wait();  // y and shared_y come from the preceding kernel
    const int vec_per_row = H >> 3;
    const size_t total = (size_t)T * vec_per_row;
    for (size_t i = blockIdx.x * (size_t)CB_THREADS + threadIdx.x; i < total;
         i += (size_t)gridDim.x * CB_THREADS) {
        const int t = (int)(i / vec_per_row);
        const int h = (int)(i - (size_t)t * vec_per_row) << 3;
        // the k rows of this token: positions and weights first, then all row pieces, so that
        // the loads of one level are in flight together
        int rows[MOE_MAX_TOPK];
        float wts[MOE_MAX_TOPK];
#pragma unroll
        for (int j = 0; j < MOE_MAX_TOPK; ++j) {
            rows[j] = j < k ? inv_perm[(size_t)t * k + j] : 0;
            wts[j] = j < k ? topk_w[(size_t)t * k + j] : 0.f;
        }
        const float s = shared_y && shared_scale ? shared_scale[t] : 1.0f;
        float acc[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
            acc[q] = 0.f;
        for (int part = 0; part < routed_parts; ++part) {
            const __nv_bfloat16 *yp = y + (size_t)part * T * k * H;
            uint4 v[MOE_MAX_TOPK];
#pragma unroll
            for (int j = 0; j < MOE_MAX_TOPK; ++j)
                if (j < k)
                    v[j] = *reinterpret_cast<const uint4 *>(yp + (size_t)rows[j] * H + h);
#pragma unroll
            for (int j = 0; j < MOE_MAX_TOPK; ++j) {
                if (j < k) {
                    const float w = wts[j];
                    acc[0] = fmaf(w, bf16_lo(v[j].x), acc[0]);
                    acc[1] = fmaf(w, bf16_hi(v[j].x), acc[1]);
                    acc[2] = fmaf(w, bf16_lo(v[j].y), acc[2]);
                    acc[3] = fmaf(w, bf16_hi(v[j].y), acc[3]);
                    acc[4] = fmaf(w, bf16_lo(v[j].z), acc[4]);
                    acc[5] = fmaf(w, bf16_hi(v[j].z), acc[5]);
                    acc[6] = fmaf(w, bf16_lo(v[j].w), acc[6]);
                    acc[7] = fmaf(w, bf16_hi(v[j].w), acc[7]);
                }
            }
        }
        if (shared_y) {
            // all planes requested before the first one is used
            uint4 sv[MOE_MAX_SHARED_PARTS];
#pragma unroll
            for (int part = 0; part < MOE_MAX_SHARED_PARTS; ++part)
                if (part < shared_parts)
                    sv[part] = *reinterpret_cast<const uint4 *>(
                        shared_y + ((size_t)part * T + t) * H + h);
#pragma unroll
            for (int part = 0; part < MOE_MAX_SHARED_PARTS; ++part) {
                if (part < shared_parts) {
                    acc[0] = fmaf(s, bf16_lo(sv[part].x), acc[0]);
                    acc[1] = fmaf(s, bf16_hi(sv[part].x), acc[1]);
                    acc[2] = fmaf(s, bf16_lo(sv[part].y), acc[2]);
                    acc[3] = fmaf(s, bf16_hi(sv[part].y), acc[3]);
                    acc[4] = fmaf(s, bf16_lo(sv[part].z), acc[4]);
                    acc[5] = fmaf(s, bf16_hi(sv[part].z), acc[5]);
                    acc[6] = fmaf(s, bf16_lo(sv[part].w), acc[6]);
                    acc[7] = fmaf(s, bf16_hi(sv[part].w), acc[7]);
                }
            }
        }
        uint4 o;
        __nv_bfloat162 p;
        p = __floats2bfloat162_rn(acc[0], acc[1]);
        o.x = *reinterpret_cast<uint32_t *>(&p);
        p = __floats2bfloat162_rn(acc[2], acc[3]);
        o.y = *reinterpret_cast<uint32_t *>(&p);
        p = __floats2bfloat162_rn(acc[4], acc[5]);
        o.z = *reinterpret_cast<uint32_t *>(&p);
        p = __floats2bfloat162_rn(acc[6], acc[7]);
        o.w = *reinterpret_cast<uint32_t *>(&p);
        *reinterpret_cast<uint4 *>(out + (size_t)t * H + h) = o;
    }
}

cudaError_t launch_combine(const moe_config_t &c, const __nv_bfloat16 *y, int routed_parts,
                           const int32_t *inv_perm, const float *topk_w,
                           const __nv_bfloat16 *shared_y, int shared_parts,
                           const float *shared_scale, int T, __nv_bfloat16 *out, cudaStream_t s)
{
    if (shared_parts > MOE_MAX_SHARED_PARTS)
        return cudaErrorInvalidValue;
    const size_t total = (size_t)T * (c.hidden >> 3);
    size_t blocks = (total + CB_THREADS - 1) / CB_THREADS;
    const size_t cap = (size_t)sm_count() * 8;
    if (blocks > cap)
        blocks = cap;
    return launch_pdl(combine_kernel, dim3((unsigned)blocks), dim3(CB_THREADS), 0, s, y, routed_parts,
                      inv_perm, topk_w, shared_y, shared_parts, shared_scale, T, c.hidden, c.top_k, out);
}

}  // namespace moe

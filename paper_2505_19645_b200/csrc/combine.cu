// Gate-weighted combine: out[t] = sum_j w[t,j] * y[inv_perm[t*K+j]] + s[t] * shared_y[t]
// (y and shared_y may arrive as partial planes, one per k chunk of the down projection).
// Gather form (each output row is summed in slot order by one owner), so the result does
// not depend on scheduling; 128-bit loads and stores.
#include "common.cuh"

namespace moe {

constexpr int CB_THREADS = 256;
constexpr int MOE_MAX_SHARED_PARTS = 8;  // k chunks of the shared expert's down pass, at most

__device__ __forceinline__ void accumulate8(float (&acc)[8], float w, const uint4 &v)
{
    acc[0] = fmaf(w, bf16_lo(v.x), acc[0]);
    acc[1] = fmaf(w, bf16_hi(v.x), acc[1]);
    acc[2] = fmaf(w, bf16_lo(v.y), acc[2]);
    acc[3] = fmaf(w, bf16_hi(v.y), acc[3]);
    acc[4] = fmaf(w, bf16_lo(v.z), acc[4]);
    acc[5] = fmaf(w, bf16_hi(v.z), acc[5]);
    acc[6] = fmaf(w, bf16_lo(v.w), acc[6]);
    acc[7] = fmaf(w, bf16_hi(v.w), acc[7]);
}

// KP: top_k rounded up to 2, 4, 8 or 16 -- the arrays of row pieces in flight are sized by it,
// so that a top-2 or top-4 layer keeps its registers (and its occupancy).
template <int KP>
__global__ void __launch_bounds__(CB_THREADS, KP <= 2 ? 4 : (KP <= 4 ? 3 : (KP <= 8 ? 2 : 1)))
combine_kernel(const __nv_bfloat16 *__restrict__ y, int routed_parts,
               const int32_t *__restrict__ inv_perm, const float *__restrict__ topk_w,
               const __nv_bfloat16 *__restrict__ shared_y, int shared_parts,
               const float *__restrict__ shared_scale, int T, int H, int k,
               __nv_bfloat16 *__restrict__ out)
{
    griddep_launch();
    griddep_wait();  // y and shared_y come from the preceding kernel
    const int vec_per_row = H >> 3;
    const size_t total = (size_t)T * vec_per_row;
    const size_t plane = (size_t)T * k * H;
    for (size_t i = blockIdx.x * (size_t)CB_THREADS + threadIdx.x; i < total;
         i += (size_t)gridDim.x * CB_THREADS) {
        const int t = (int)(i / vec_per_row);
        const int h = (int)(i - (size_t)t * vec_per_row) << 3;
        // the k rows of this token: positions and weights first, then the row pieces of a
        // plane, so that the loads of one level are in flight together
        int rows[KP];
        float wts[KP];
#pragma unroll
        for (int j = 0; j < KP; ++j) {
            rows[j] = j < k ? inv_perm[(size_t)t * k + j] : 0;
            wts[j] = j < k ? topk_w[(size_t)t * k + j] : 0.f;
        }
        const float s = shared_y && shared_scale ? shared_scale[t] : 1.0f;
        // the shared expert's planes, four at a time, requested before the routed rows are used
        uint4 sv[4];
        const int sp0 = shared_y ? (shared_parts < 4 ? shared_parts : 4) : 0;
#pragma unroll
        for (int p = 0; p < 4; ++p)
            if (p < sp0)
                sv[p] = *reinterpret_cast<const uint4 *>(shared_y + ((size_t)p * T + t) * H + h);
        float acc[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
            acc[q] = 0.f;
        for (int part = 0; part < routed_parts; ++part) {
            const __nv_bfloat16 *yp = y + (size_t)part * plane;
            uint4 v[KP];
#pragma unroll
            for (int j = 0; j < KP; ++j)
                if (j < k)
                    v[j] = *reinterpret_cast<const uint4 *>(yp + (size_t)rows[j] * H + h);
#pragma unroll
            for (int j = 0; j < KP; ++j)
                if (j < k)
                    accumulate8(acc, wts[j], v[j]);
        }
#pragma unroll
        for (int p = 0; p < 4; ++p)
            if (p < sp0)
                accumulate8(acc, s, sv[p]);
        if (shared_y && shared_parts > 4) {
#pragma unroll
            for (int p = 0; p < 4; ++p)
                if (4 + p < shared_parts)
                    sv[p] = *reinterpret_cast<const uint4 *>(
                        shared_y + ((size_t)(4 + p) * T + t) * H + h);
#pragma unroll
            for (int p = 0; p < 4; ++p)
                if (4 + p < shared_parts)
                    accumulate8(acc, s, sv[p]);
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
#define MOE_CB_LAUNCH(KP)                                                                        \
    return launch_pdl(combine_kernel<KP>, dim3((unsigned)blocks), dim3(CB_THREADS), 0, s, y,     \
                      routed_parts, inv_perm, topk_w, shared_y, shared_parts, shared_scale, T,   \
                      c.hidden, c.top_k, out)
    if (c.top_k <= 2)
        MOE_CB_LAUNCH(2);
    if (c.top_k <= 4)
        MOE_CB_LAUNCH(4);
    if (c.top_k <= 8)
        MOE_CB_LAUNCH(8);
    MOE_CB_LAUNCH(16);
#undef MOE_CB_LAUNCH
}

}  // namespace moe

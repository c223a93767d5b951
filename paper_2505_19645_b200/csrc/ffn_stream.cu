// Streaming (GEMV-style) expert FFN for groups with few rows: every weight element is
// loaded from HBM exactly once with 128-bit loads straight into registers, and applied to
// up to 32 token rows at once.  The multiply-accumulate of the 8 bf16 values a lane holds
// against the token rows is issued as warp-level m16n8k16 MMAs (fp32 accumulate), so 1..8
// rows cost the same as one; the data flow stays that of a matrix-vector product: no
// shared-memory staging of weights, no reuse of a weight tile.
//
// Work decomposition: a persistent grid walks the items (segment, row block).  Within a
// CTA of 8 warps, 2 row tiles x 4 K-slices; the K-slices are summed through shared memory.
#include "common.cuh"

namespace moe {

constexpr int ST_THREADS = 256;
constexpr int ST_KS = 4;  // K slices per row tile (warps)
constexpr int ST_MT = 2;  // row-tile pairs per CTA
constexpr int ST_MAX_NCH = SEG_TOKENS / 8;

struct StreamArgs {
    // [group][...]: 0 = routed experts, 1 = shared expert
    const __nv_bfloat16 *wa[2];  // gated: W_gate [*, rows, K]; down: W_down [*, rows, K]
    const __nv_bfloat16 *wb[2];  // gated: W_up; down: unused
    int rows[2];                 // output features per group: I / I_s (gated) or H (down)
    int K[2];                    // reduction length: H (gated) or I / I_s (down)
    const __nv_bfloat16 *in[2];  // gated: x [T,H]; down: h [A,I] / h_shared [T,I_s]
    __nv_bfloat16 *out[2];       // gated: h / h_shared; down: y / y_shared
    const int32_t *perm;         // gated, routed: token of sorted row r is perm[r] / top_k
    int top_k;
    const int32_t *plan_header;
    const Segment *seg[2];
};

// One warp: two 16-row A tiles (pointers pre-offset to this lane's row and 8-element k
// group) against NCH chunks of 8 token rows, over k-steps [s0, s1) of 32 elements.
//
// A lane holding 8 consecutive k values of row g (and of row g+8) feeds two MMAs by
// re-labelling k inside the 32-wide step: MMA #1 contracts the physical k positions
// 8t+{0,1,2,3}, MMA #2 the positions 8t+{4,5,6,7}; the B fragment is loaded with the same
// labelling, and a contraction does not care about the order of k.
template <int NCH>
__device__ __forceinline__ void stream_tiles(const __nv_bfloat16 *a0lo, const __nv_bfloat16 *a0hi,
                                             const __nv_bfloat16 *a1lo, const __nv_bfloat16 *a1hi,
                                             const __nv_bfloat16 *(&b)[ST_MAX_NCH], int s0, int s1,
                                             float (&acc)[2][ST_MAX_NCH][4])
{
    int s = s0;
    for (; s + 2 <= s1; s += 2) {
        uint4 A[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int k = (s + u) * 32;
            A[u][0] = ld_stream_v4(a0lo + k);
            A[u][1] = ld_stream_v4(a0hi + k);
            A[u][2] = ld_stream_v4(a1lo + k);
            A[u][3] = ld_stream_v4(a1hi + k);
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int k = (s + u) * 32;
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const uint4 B = ld_cached_v4(b[c] + k);
                mma_bf16_16816(acc[0][c], A[u][0].x, A[u][1].x, A[u][0].y, A[u][1].y, B.x, B.y);
                mma_bf16_16816(acc[0][c], A[u][0].z, A[u][1].z, A[u][0].w, A[u][1].w, B.z, B.w);
                mma_bf16_16816(acc[1][c], A[u][2].x, A[u][3].x, A[u][2].y, A[u][3].y, B.x, B.y);
                mma_bf16_16816(acc[1][c], A[u][2].z, A[u][3].z, A[u][2].w, A[u][3].w, B.z, B.w);
            }
        }
    }
    for (; s < s1; ++s) {
        const int k = s * 32;
        const uint4 A0 = ld_stream_v4(a0lo + k), A1 = ld_stream_v4(a0hi + k);
        const uint4 A2 = ld_stream_v4(a1lo + k), A3 = ld_stream_v4(a1hi + k);
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
            const uint4 B = ld_cached_v4(b[c] + k);
            mma_bf16_16816(acc[0][c], A0.x, A1.x, A0.y, A1.y, B.x, B.y);
            mma_bf16_16816(acc[0][c], A0.z, A1.z, A0.w, A1.w, B.z, B.w);
            mma_bf16_16816(acc[1][c], A2.x, A3.x, A2.y, A3.y, B.x, B.y);
            mma_bf16_16816(acc[1][c], A2.z, A3.z, A2.w, A3.w, B.z, B.w);
        }
    }
}

// GATED: rows of W_gate and W_up -> h = silu(g) * u.   !GATED: rows of W_down -> y.
template <bool GATED>
__global__ void __launch_bounds__(ST_THREADS, 2) ffn_stream_kernel(const StreamArgs args)
{
    // partial sums: [k-slice][row-tile pair][tile][chunk][acc reg][lane]
    __shared__ float part[ST_KS][ST_MT][2][ST_MAX_NCH][4][32];

    constexpr int RB = GATED ? ST_MT * 16 : ST_MT * 32;  // output rows per CTA item
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int mt = warp / ST_KS, ks = warp % ST_KS;

    const int nseg0 = args.plan_header[0], nseg1 = args.plan_header[1];
    const int nrb0 = (args.rows[0] + RB - 1) / RB;
    const int nrb1 = nseg1 > 0 ? (args.rows[1] + RB - 1) / RB : 0;
    const int items0 = nseg0 * nrb0;
    const int items = items0 + nseg1 * nrb1;

    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        // row-block major: the segments of one expert's row block are neighbours in time
        int grp, rb, si;
        if (item < items0) {
            grp = 0;
            rb = item / nseg0;
            si = item - rb * nseg0;
        } else {
            grp = 1;
            const int w = item - items0;
            rb = w / nseg1;
            si = w - rb * nseg1;
        }
        const Segment sg = args.seg[grp][si];
        const int rows = args.rows[grp], K = args.K[grp];
        const int n = sg.n;
        const int nch = (n + 7) >> 3;
        const size_t wbase = grp == 0 ? (size_t)sg.expert * rows * K : 0;

        // this lane's A row pointers (clamped rows are computed and dropped)
        const int r0 = rb * RB + mt * (GATED ? 16 : 32);
        const __nv_bfloat16 *a0lo, *a0hi, *a1lo, *a1hi;
        {
            const int last = rows - 1;
            const __nv_bfloat16 *wa = args.wa[grp] + wbase + 8 * tq;
            if (GATED) {
                const __nv_bfloat16 *wb = args.wb[grp] + wbase + 8 * tq;
                a0lo = wa + (size_t)min(r0 + g, last) * K;
                a0hi = wa + (size_t)min(r0 + g + 8, last) * K;
                a1lo = wb + (size_t)min(r0 + g, last) * K;
                a1hi = wb + (size_t)min(r0 + g + 8, last) * K;
            } else {
                a0lo = wa + (size_t)min(r0 + g, last) * K;
                a0hi = wa + (size_t)min(r0 + g + 8, last) * K;
                a1lo = wa + (size_t)min(r0 + 16 + g, last) * K;
                a1hi = wa + (size_t)min(r0 + 24 + g, last) * K;
            }
        }
        // this lane's B row pointers: token row (chunk c, slot g)
        const __nv_bfloat16 *b[ST_MAX_NCH];
#pragma unroll
        for (int c = 0; c < ST_MAX_NCH; ++c) {
            const int slot = min(c * 8 + g, n - 1);
            int src = sg.row0 + slot;
            if (GATED && grp == 0)
                src = args.perm[src] / args.top_k;
            b[c] = args.in[grp] + (size_t)src * K + 8 * tq;
        }

        float acc[2][ST_MAX_NCH][4];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int c = 0; c < ST_MAX_NCH; ++c)
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    acc[i][c][q] = 0.f;

        const int nsteps = K >> 5;
        const int s0 = (int)((long long)ks * nsteps / ST_KS);
        const int s1 = (int)((long long)(ks + 1) * nsteps / ST_KS);
        switch (nch) {
        case 1: stream_tiles<1>(a0lo, a0hi, a1lo, a1hi, b, s0, s1, acc); break;
        case 2: stream_tiles<2>(a0lo, a0hi, a1lo, a1hi, b, s0, s1, acc); break;
        case 3: stream_tiles<3>(a0lo, a0hi, a1lo, a1hi, b, s0, s1, acc); break;
        default: stream_tiles<4>(a0lo, a0hi, a1lo, a1hi, b, s0, s1, acc); break;
        }

#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int c = 0; c < ST_MAX_NCH; ++c)
                if (c < nch) {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        part[ks][mt][i][c][q][lane] = acc[i][c][q];
                }
        __syncthreads();

        // Epilogue over (token slot, output row) with the row fastest across threads.
        // Accumulator register q of lane (g,tq) in chunk c is row g + 8*(q>>1) of the tile
        // and token slot c*8 + 2*tq + (q&1).
        __nv_bfloat16 *out = args.out[grp];
        const int n_out = RB * n;
        for (int o = tid; o < n_out; o += ST_THREADS) {
            const int r = o % RB, slot = o / RB;
            const int c = slot >> 3, tt = (slot & 7) >> 1, lo = slot & 1;
            int pm, tile, rr;
            if (GATED) {
                pm = r >> 4;
                tile = 0;
                rr = r & 15;
            } else {
                pm = r >> 5;
                tile = (r >> 4) & 1;
                rr = r & 15;
            }
            const int q = ((rr >> 3) << 1) | lo;
            const int ln = ((rr & 7) << 2) | tt;
            const int row = rb * RB + r;
            if (row >= rows)
                continue;
            float v0 = 0.f, v1 = 0.f;
#pragma unroll
            for (int s = 0; s < ST_KS; ++s) {
                v0 += part[s][pm][tile][c][q][ln];
                if (GATED)
                    v1 += part[s][pm][1][c][q][ln];
            }
            const float res = GATED ? silu_f(v0) * v1 : v0;
            out[(size_t)(sg.row0 + slot) * rows + row] = __float2bfloat16(res);
        }
        __syncthreads();
    }
}

static int stream_grid(int max_items)
{
    const int resident = sm_count() * 2;
    return max_items < resident ? (max_items > 0 ? max_items : 1) : resident;
}

cudaError_t launch_ffn_stream_gateup(const moe_config_t &c, const moe_weights_t &w,
                                     const __nv_bfloat16 *x, int T, const int32_t *perm,
                                     PlanView plan, bool with_shared, __nv_bfloat16 *h,
                                     __nv_bfloat16 *h_shared, cudaStream_t s)
{
    StreamArgs a{};
    a.wa[0] = static_cast<const __nv_bfloat16 *>(w.w_gate);
    a.wb[0] = static_cast<const __nv_bfloat16 *>(w.w_up);
    a.wa[1] = static_cast<const __nv_bfloat16 *>(w.ws_gate);
    a.wb[1] = static_cast<const __nv_bfloat16 *>(w.ws_up);
    a.rows[0] = c.inter;
    a.rows[1] = c.shared_inter;
    a.K[0] = a.K[1] = c.hidden;
    a.in[0] = a.in[1] = x;
    a.out[0] = h;
    a.out[1] = h_shared;
    a.perm = perm;
    a.top_k = c.top_k;
    a.plan_header = plan.header;
    a.seg[0] = plan.routed;
    a.seg[1] = plan.shared;
    constexpr int RB = ST_MT * 16;
    const int A = T * c.top_k;
    long long items = (long long)max_routed_segments(c.n_experts, A) * ((c.inter + RB - 1) / RB);
    if (with_shared)
        items += (long long)max_shared_segments(T) * ((c.shared_inter + RB - 1) / RB);
    ffn_stream_kernel<true><<<stream_grid((int)(items > (1 << 30) ? (1 << 30) : items)),
                              ST_THREADS, 0, s>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_ffn_stream_down(const moe_config_t &c, const moe_weights_t &w, int T,
                                   PlanView plan, bool with_shared, const __nv_bfloat16 *h,
                                   const __nv_bfloat16 *h_shared, __nv_bfloat16 *y,
                                   __nv_bfloat16 *y_shared, cudaStream_t s)
{
    StreamArgs a{};
    a.wa[0] = static_cast<const __nv_bfloat16 *>(w.w_down);
    a.wa[1] = static_cast<const __nv_bfloat16 *>(w.ws_down);
    a.wb[0] = a.wb[1] = nullptr;
    a.rows[0] = a.rows[1] = c.hidden;
    a.K[0] = c.inter;
    a.K[1] = c.shared_inter;
    a.in[0] = h;
    a.in[1] = h_shared;
    a.out[0] = y;
    a.out[1] = y_shared;
    a.perm = nullptr;
    a.top_k = c.top_k;
    a.plan_header = plan.header;
    a.seg[0] = plan.routed;
    a.seg[1] = plan.shared;
    constexpr int RB = ST_MT * 32;
    const int A = T * c.top_k;
    long long items = (long long)max_routed_segments(c.n_experts, A) * ((c.hidden + RB - 1) / RB);
    if (with_shared)
        items += (long long)max_shared_segments(T) * ((c.hidden + RB - 1) / RB);
    ffn_stream_kernel<false><<<stream_grid((int)(items > (1 << 30) ? (1 << 30) : items)),
                               ST_THREADS, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace moe

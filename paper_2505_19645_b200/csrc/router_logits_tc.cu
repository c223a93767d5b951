// Router logits for large batches on the 5th-generation tensor cores.
//
//   z[t,e] = x[t,:] . w_router[e,:] (+ bias[e]),   s[t] = sigmoid(x[t,:] . w_sg)
//
// with fp32-level accuracy from bf16 instructions: every fp32 router row is split once per call
// into three bf16 rows  w = hi + mid + lo  (each remainder is exact in fp32, so the three carry
// 24 mantissa bits; the bf16 token values are exact) and the three products are accumulated in
// the same fp32 accumulator in TMEM.  Two kernels here, and the first step of a third:
//   split   w_router (and the bf16 gate vector) -> planes [3][R][H] bf16, R = E (+1)
//   gemm    one CTA per (256 tokens, 256 router rows, k chunk): TMA -> shared-memory rings ->
//           tcgen05.mma (router rows as M, two blocks of 128; tokens as N) -> partial sums
//           [S][T][R] fp32
//   sum     route_topk_sum_kernel (router.cu): the warp that ranks a token's logits first adds its
//           S partial rows in chunk order, adds the bias and applies the gate's sigmoid
// The reduction over H is cut into S chunks so that about one CTA per SM has work even when
// there are only a dozen token tiles; the partial planes are summed in chunk order, so the
// logits do not depend on timing.  Used for large batches (router_logits_tc_applies), where the
// mma.sync kernel of router_logits.cu, which splits the rows on the fly for every token tile,
// takes 60-300 us.
#include <string.h>

#include <mutex>

#include "tc_ptx.cuh"

namespace moe {

constexpr int RT_THREADS = 192;       // producer, MMA issuer, four epilogue warps
constexpr int RT_TOKENS = 256;        // token rows per CTA (the instruction's N)
constexpr int RT_A_SLOTS = 4;         // ring of 32 KB slots: one plane of one k box, 2 x 128 rows
constexpr int RT_B_SLOTS = 2;         // ring of 32 KB entries: 256 token rows of one k box
constexpr int RT_A_BYTES = 2 * 128 * 128;
constexpr int RT_B_BYTES = RT_TOKENS * 128;
constexpr int RT_MAX_SPLIT = 16;
constexpr int RT_SMEM = RT_A_SLOTS * RT_A_BYTES + RT_B_SLOTS * RT_B_BYTES + 1024;

// From about 128 K logits on the mma.sync kernel takes longer than the launches here
// (measured: 256 experts from 512 tokens, 64 experts from 2048 tokens).
bool router_logits_tc_applies(const moe_config_t &c, int T)
{
    return T >= 512 && (long long)T * c.n_experts >= 128 * 1024 && c.hidden >= 512;
}

static int router_rows(const moe_config_t &c)
{
    return c.n_experts + ((c.shared_gate && c.shared_inter > 0) ? 1 : 0);
}

// k chunks: about one CTA per SM, at least four 64-element boxes per chunk
static int router_split(const moe_config_t &c, int T)
{
    const int tiles = (T + RT_TOKENS - 1) / RT_TOKENS * ((router_rows(c) + 255) / 256);
    const int boxes = (c.hidden + 63) / 64;
    int s = sm_count() / tiles;
    if (s > boxes / 4)
        s = boxes / 4;
    if (s > RT_MAX_SPLIT)
        s = RT_MAX_SPLIT;
    return s < 1 ? 1 : s;
}

size_t router_tc_plane_bytes(const moe_config_t &c, int T)
{
    return router_logits_tc_applies(c, T) ? (size_t)3 * router_rows(c) * c.hidden * 2 : 0;
}

size_t router_tc_partial_bytes(const moe_config_t &c, int T)
{
    return router_logits_tc_applies(c, T) ? (size_t)RT_MAX_SPLIT * T * router_rows(c) * 4 : 0;
}

// ---- split: fp32 router rows -> three bf16 planes ---------------------------------------------

__device__ __forceinline__ uint32_t rt_pack2(float a, float b)
{
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&p);
}

// planes[p][r][h]: p = 0 hi, 1 mid, 2 lo; rows r < E from w_router, row E (if present) the bf16
// gate vector (exact in the hi plane).  First kernel of a layer call: also clears the counters
// a later kernel of the call updates before the plan exists, and initialises the status region.
__global__ void __launch_bounds__(256)
router_split_kernel(const float *__restrict__ w_router, const __nv_bfloat16 *__restrict__ w_sg, int E,
                    int R, int H, __nv_bfloat16 *__restrict__ planes, int32_t *__restrict__ zero,
                    int zero_n, int32_t *__restrict__ status)
{
    griddep_wait();  // first kernel of a layer call: everything older is complete from here on
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < zero_n; i += blockDim.x)
            zero[i] = 0;
        if (threadIdx.x == 0)
            status_region_init(status);
        __threadfence();
        __syncthreads();
    }
    griddep_launch();
    const size_t plane = (size_t)R * H;
    const size_t n8 = plane >> 3;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n8;
         i += (size_t)gridDim.x * blockDim.x) {
        const size_t at = i << 3;
        const int r = (int)(at / H);
        uint4 hi, mid, lo;
        if (r < E) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(w_router + at));
            const float4 b = __ldg(reinterpret_cast<const float4 *>(w_router + at + 4));
            const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
            uint32_t h[4], m[4], l[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                h[j] = rt_pack2(v[2 * j], v[2 * j + 1]);
                const float ra = v[2 * j] - bf16_lo(h[j]), rb = v[2 * j + 1] - bf16_hi(h[j]);
                m[j] = rt_pack2(ra, rb);
                l[j] = rt_pack2(ra - bf16_lo(m[j]), rb - bf16_hi(m[j]));
            }
            hi = make_uint4(h[0], h[1], h[2], h[3]);
            mid = make_uint4(m[0], m[1], m[2], m[3]);
            lo = make_uint4(l[0], l[1], l[2], l[3]);
        } else {
            hi = __ldg(reinterpret_cast<const uint4 *>(w_sg + (at - (size_t)E * H)));
            mid = lo = make_uint4(0u, 0u, 0u, 0u);
        }
        *reinterpret_cast<uint4 *>(planes + at) = hi;
        *reinterpret_cast<uint4 *>(planes + plane + at) = mid;
        *reinterpret_cast<uint4 *>(planes + 2 * plane + at) = lo;
    }
}

// ---- gemm -----------------------------------------------------------------------------------------

struct RouterTcArgs {
    int T, R, H;
    int token_tiles, row_pairs, split;  // grid = token_tiles * row_pairs * split
    float *partial;                     // [split][T][R]
    int32_t *status;
    int wait_us;
};

struct RouterTcMaps {
    CUtensorMap planes;  // [3 * R, H] bf16, box 64 x 128
    CUtensorMap x;       // [T, H] bf16, box 64 x 128
};

// One CTA = one (token tile, pair of 128-row blocks, k chunk).  warp 0: producer (one lane
// issues the TMA loads of both rings), warp 1: MMA issuer and owner of the TMEM allocation,
// warps 2..5: epilogue (a lane is a router row, a column a token; 32 lanes store 128 contiguous
// bytes of a token's partial logits).  Rows beyond R and tokens beyond T are zero-filled by TMA
// or belong to the next plane; they are computed and never stored.
__global__ void __launch_bounds__(RT_THREADS, 1)
router_logits_tc_kernel(const RouterTcArgs args, const __grid_constant__ RouterTcMaps maps)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * RT_A_SLOTS + 2 * RT_B_SLOTS + 1];
    __shared__ uint32_t tmem_base_holder;
    __shared__ int abort_flag[2];

    const uint32_t ring_b = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t ring_a = ring_b + RT_B_SLOTS * RT_B_BYTES;
    const uint32_t bar0 = smem_u32(bars);
    auto a_full = [&](int s) { return bar0 + 8u * s; };
    auto a_empty = [&](int s) { return bar0 + 8u * (RT_A_SLOTS + s); };
    auto b_full = [&](int s) { return bar0 + 8u * (2 * RT_A_SLOTS + s); };
    auto b_empty = [&](int s) { return bar0 + 8u * (2 * RT_A_SLOTS + RT_B_SLOTS + s); };
    const uint32_t acc_full = bar0 + 8u * (2 * RT_A_SLOTS + 2 * RT_B_SLOTS);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag[0] = 0;
        abort_flag[1] = args.wait_us;
        for (int s = 0; s < RT_A_SLOTS; ++s) {
            mbar_init(a_full(s), 1);
            mbar_init(a_empty(s), 1);
        }
        for (int s = 0; s < RT_B_SLOTS; ++s) {
            mbar_init(b_full(s), 1);
            mbar_init(b_empty(s), 1);
        }
        mbar_init(acc_full, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        prefetch_map(&maps.planes);
        prefetch_map(&maps.x);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(&tmem_base_holder)),
                     "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_holder;
    volatile int *abortp = abort_flag;

    // this CTA's item
    const int item = blockIdx.x;
    const int chunk = item % args.split;
    const int pair = (item / args.split) % args.row_pairs;
    const int tile = item / (args.split * args.row_pairs);
    const int t0 = tile * RT_TOKENS;
    const int n = min(RT_TOKENS, args.T - t0);
    const int npad = (n + 15) & ~15;
    const int boxes = (args.H + 63) >> 6;
    const int kb0 = chunk * boxes / args.split, kb1 = (chunk + 1) * boxes / args.split;
    const int row0 = pair * 256;
    const int nblk = args.R - row0 > 128 ? 2 : 1;

    griddep_launch();
    if (warp == 0) {
        if (lane == 0) {
            griddep_wait();  // the planes come from the preceding kernel
            const uint64_t keep = l2_policy_evict_last();
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            bool ok = true;
            for (int kb = kb0; ok && kb < kb1; ++kb) {
                if (!mbar_wait(b_empty(sb), pb ^ 1u, abortp, args.status))
                    break;
                const uint32_t bdst = ring_b + sb * RT_B_BYTES;
                // (a box is always transferred whole: rows beyond T arrive as zeros)
                mbar_expect_tx(b_full(sb), (uint32_t)((npad + 127) >> 7) * 128u * 128u);
                // the token rows as boxes of 128 rows (the tensor map's box); a partial tile
                // takes what it needs, rounded up to whole boxes of its map
                for (int r = 0; r < npad; r += 128)
                    tma_load_2d_hint(bdst + r * 128, &maps.x, b_full(sb), kb * 64, t0 + r, keep);
                if (++sb == RT_B_SLOTS) {
                    sb = 0;
                    pb ^= 1u;
                }
                for (int p = 2; ok && p >= 0; --p) {  // lo, mid, hi: small terms first
                    if (!mbar_wait(a_empty(sa), pa ^ 1u, abortp, args.status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t adst = ring_a + sa * RT_A_BYTES;
                    mbar_expect_tx(a_full(sa), (uint32_t)nblk * 128u * 128u);
                    for (int b = 0; b < nblk; ++b)
                        tma_load_2d_hint(adst + b * 128 * 128, &maps.planes, a_full(sa), kb * 64,
                                         p * args.R + row0 + 128 * b, keep);
                    if (++sa == RT_A_SLOTS) {
                        sa = 0;
                        pa ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(npad);
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            bool ok = true;
            for (int kb = kb0; ok && kb < kb1; ++kb) {
                if (!mbar_wait(b_full(sb), pb, abortp, args.status))
                    break;
                const uint64_t x_desc = umma_desc_sw128(ring_b + sb * RT_B_BYTES);
                for (int p = 0; p < 3; ++p) {
                    if (!mbar_wait(a_full(sa), pa, abortp, args.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint64_t w_desc = umma_desc_sw128(ring_a + sa * RT_A_BYTES);
                    const uint32_t accum = (kb != kb0 || p != 0) ? 1u : 0u;
                    if (nblk == 2)
                        issue_k_box<2>(tmem_base, 256u, w_desc, (128u * 128u) >> 4, x_desc, idesc, accum);
                    else
                        issue_k_box<1>(tmem_base, 256u, w_desc, (128u * 128u) >> 4, x_desc, idesc, accum);
                    umma_commit(a_empty(sa));
                    if (++sa == RT_A_SLOTS) {
                        sa = 0;
                        pa ^= 1u;
                    }
                }
                if (!ok)
                    break;
                umma_commit(b_empty(sb));
                if (++sb == RT_B_SLOTS) {
                    sb = 0;
                    pb ^= 1u;
                }
            }
            if (ok)
                umma_commit(acc_full);
        }
    } else {
        const int quarter = warp & 3;  // TMEM lanes 32 * quarter .. + 31
        const bool ready = mbar_wait(acc_full, 0u, abortp, args.status);
        if (__all_sync(0xffffffffu, ready)) {
            tc_fence_after();
            for (int b = 0; b < nblk; ++b) {
                const int e = row0 + 128 * b + quarter * 32 + lane;
                if (row0 + 128 * b + quarter * 32 >= args.R)
                    break;  // (uniform) this warp's rows lie beyond the last router row
                float *out = args.partial + ((size_t)chunk * args.T + t0) * args.R + e;
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + 256u * b;
                for (int c = 0; c < npad; c += 16) {
                    uint32_t v[16];
                    tmem_ld16(taddr + c, v);
                    tmem_ld_wait();
                    if (e < args.R) {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (c + i < n)
                                out[(size_t)(c + i) * args.R] = __uint_as_float(v[i]);
                    }
                }
            }
        }
    }

    if (*abortp) {
        // a wait gave up: hold the CTA until copies and instructions in flight have landed
        const uint64_t t_hold = global_ns();
        while (global_ns() - t_hold < 1000000ull) {
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512)
                     : "memory");
    }
    griddep_wait();  // no kernel of the chain completes before its predecessor
}

// ---- host -----------------------------------------------------------------------------------------

cudaError_t launch_router_logits_tc(const moe_config_t &c, const moe_weights_t &w,
                                    const __nv_bfloat16 *x, int T, __nv_bfloat16 *planes,
                                    float *partial, cudaStream_t s, int32_t *zero, int zero_n,
                                    int32_t *status, int *launches, int *chunks)
{
    const int E = c.n_experts, R = router_rows(c), H = c.hidden;
    cudaError_t err = launch_pdl(router_split_kernel, dim3(2 * sm_count()), dim3(256), 0, s, w.w_router,
                                 static_cast<const __nv_bfloat16 *>(w.w_shared_gate), E, R, H, planes,
                                 zero, zero_n, status);
    if (err != cudaSuccess)
        return err;
    ++*launches;

    RouterTcArgs a{};
    a.T = T;
    a.R = R;
    a.H = H;
    a.token_tiles = (T + RT_TOKENS - 1) / RT_TOKENS;
    a.row_pairs = (R + 255) / 256;
    a.split = router_split(c, T);
    a.partial = partial;
    a.status = status;
    a.wait_us = (int)(FF_WAIT_NS / 1000ull);
    // tensor maps: kept per (device, pointers, extents) like the FFN kernels' (a few entries)
    struct Key {
        int device;
        const void *planes, *x;
        int T, R, H;
    };
    struct Entry {
        bool used;
        Key key;
        RouterTcMaps maps;
    };
    static Entry cache[8];
    static int next = 0;
    static std::mutex mutex;
    Key key;
    memset(&key, 0, sizeof key);
    cudaGetDevice(&key.device);
    key.planes = planes;
    key.x = x;
    key.T = T;
    key.R = R;
    key.H = H;
    RouterTcMaps maps;
    bool hit = false;
    {
        std::lock_guard<std::mutex> lock(mutex);
        for (const Entry &e : cache)
            if (e.used && memcmp(&e.key, &key, sizeof key) == 0) {
                maps = e.maps;
                hit = true;
                break;
            }
    }
    if (!hit) {
        if (!make_tma_map_2d_bf16(&maps.planes, planes, (uint64_t)3 * R, H, 128) ||
            !make_tma_map_2d_bf16(&maps.x, x, T, H, 128))
            return cudaErrorInvalidValue;
        std::lock_guard<std::mutex> lock(mutex);
        cache[next] = Entry{true, key, maps};
        next = (next + 1) % 8;
    }
    static DeviceOnce configured;
    if (!configured.done(key.device)) {
        err = cudaFuncSetAttribute(router_logits_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   RT_SMEM);
        if (err != cudaSuccess)
            return err;
        configured.mark(key.device);
    }
    err = launch_pdl(router_logits_tc_kernel, dim3(a.token_tiles * a.row_pairs * a.split),
                     dim3(RT_THREADS), RT_SMEM, s, a, maps);
    if (err != cudaSuccess)
        return err;
    ++*launches;

    *chunks = a.split;  // the caller's top-k kernel sums them
    return cudaSuccess;
}

}  // namespace moe

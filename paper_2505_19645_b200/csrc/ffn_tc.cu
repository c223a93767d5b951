// Tensor-core expert FFN for groups with many token rows: tcgen05.mma with the accumulator
// in TMEM, operands staged in shared memory by TMA (128-byte swizzle), fp32 accumulation.
//
// The contraction is issued "swapped": the 128 rows of a weight tile are the MMA's M, the
// group's token rows are its N (16..128), both operands K-major.  A weight tile is thus
// streamed from HBM exactly once per (group, 128-row block) whatever the token count, and a
// group with few tokens still fills the instruction.
//
// CTA = 6 warps: warp 0 issues TMA loads (one elected lane), warp 1 owns TMEM and issues the
// MMAs (one lane), warps 2..5 read the accumulators back (tcgen05.ld, one TMEM lane quarter
// each), apply SwiGLU / nothing, and store bf16.  A ring of shared-memory stages connects
// producer and MMA warp, two accumulator buffers connect MMA warp and epilogue, all through
// mbarriers.  Every wait is bounded: when a wait gives up it raises the CTA's abort flag and
// the device status word, every role leaves its loop, TMEM is freed and the kernel returns.
#include <cuda.h>
#include <string.h>

#include "common.cuh"

namespace moe {

constexpr int TC_M = 128;          // weight rows per tile (UMMA M)
constexpr int TC_KB = 64;          // K elements per stage: one 128-byte swizzle row
constexpr int TC_THREADS = 192;
constexpr int TC_STAGES_GATED = 4;  // 4 x 48 KB
constexpr int TC_STAGES_DOWN = 6;   // 6 x 32 KB
constexpr uint32_t TC_TILE_BYTES = TC_M * TC_KB * 2;  // 16 KB, also the B tile (128 rows)
constexpr uint64_t TC_WAIT_NS = 1000ull * 1000ull * 1000ull;  // 1 s per wait
constexpr int TC_TMEM_COLS = 512;

struct TcArgs {
    int rows[2];      // output features per group kind (routed, shared)
    int K[2];         // reduction length per group kind
    __nv_bfloat16 *out[2];
    int out_ld[2];
    const int32_t *plan_header;
    const Segment *seg[2];
    int32_t *status;
};

// ---- PTX wrappers ----------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t global_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false (and raises the abort flag) if the phase did not complete in
// TC_WAIT_NS or another role already aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          int32_t *status)
{
    if (mbar_try_wait(bar, parity))
        return true;
    const uint64_t t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity))
                return true;
        if (*abort_flag)
            return false;
        if (global_ns() - t0 > TC_WAIT_NS) {
            *abort_flag = 1;
            atomicExch(status, 1);
            return false;
        }
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                            int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4}], [%2];"
        :
        : "r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :
        : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Arrives on the mbarrier when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15])
        : "r"(taddr));
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) with
// the 128-byte swizzle TMA wrote: 8-row groups 1024 bytes apart (stride byte offset), leading
// byte offset unused for swizzled K-major (1), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}

// kind::f16 instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(TC_M >> 4) << 24);
}

// ---- kernel ----------------------------------------------------------------------------

template <bool GATED>
__global__ void __launch_bounds__(TC_THREADS, 1)
ffn_tc_kernel(const TcArgs args, const __grid_constant__ CUtensorMap map_a0_r,
              const __grid_constant__ CUtensorMap map_a1_r,
              const __grid_constant__ CUtensorMap map_b_r,
              const __grid_constant__ CUtensorMap map_a0_s,
              const __grid_constant__ CUtensorMap map_a1_s,
              const __grid_constant__ CUtensorMap map_b_s)
{
    constexpr int STAGES = GATED ? TC_STAGES_GATED : TC_STAGES_DOWN;
    constexpr int NA = GATED ? 2 : 1;                       // weight tiles per stage
    constexpr uint32_t STAGE_BYTES = (NA + 1) * TC_TILE_BYTES;
    constexpr int ACC_COLS = GATED ? 256 : 128;             // TMEM columns per accumulator buffer

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * STAGES + 4];
    __shared__ uint32_t tmem_base_holder;
    __shared__ int abort_flag;

    const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle needs 1 KB alignment
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto accf_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
    auto acce_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int nseg0 = args.plan_header[2], nseg1 = args.plan_header[3];
    const int nmt0 = (args.rows[0] + TC_M - 1) / TC_M;
    const int nmt1 = nseg1 > 0 ? (args.rows[1] + TC_M - 1) / TC_M : 0;
    const int items0 = nseg0 * nmt0;
    const int items = items0 + nseg1 * nmt1;
    if ((int)blockIdx.x >= items)
        return;  // uniform for the CTA, before any barrier or TMEM use

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(accf_bar(b), 1);
            mbar_init(acce_bar(b), 4);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(&tmem_base_holder)),
                     "r"(TC_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_holder;
    volatile int *abortp = &abort_flag;

    // decode of work item -> (group kind, segment, row tile); row-tile major so that the
    // segments sharing a weight tile run next to each other
    auto decode = [&](int item, int &grp, int &mt, Segment &sg) {
        int si;
        if (item < items0) {
            grp = 0;
            mt = item / nseg0;
            si = item - mt * nseg0;
        } else {
            grp = 1;
            const int w = item - items0;
            mt = w / nseg1;
            si = w - mt * nseg1;
        }
        sg = args.seg[grp][si];
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < items; item += gridDim.x) {
                int grp, mt;
                Segment sg;
                decode(item, grp, mt, sg);
                const CUtensorMap *ma0 = grp == 0 ? &map_a0_r : &map_a0_s;
                const CUtensorMap *ma1 = grp == 0 ? &map_a1_r : &map_a1_s;
                const CUtensorMap *mb = grp == 0 ? &map_b_r : &map_b_s;
                const int wrow = (grp == 0 ? sg.expert * args.rows[0] : 0) + mt * TC_M;
                const int nkb = (args.K[grp] + TC_KB - 1) / TC_KB;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp, args.status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t base = tiles + stage * STAGE_BYTES;
                    mbar_expect_tx(full_bar(stage), STAGE_BYTES);
                    tma_load_2d(base, ma0, full_bar(stage), kb * TC_KB, wrow);
                    if (GATED)
                        tma_load_2d(base + TC_TILE_BYTES, ma1, full_bar(stage), kb * TC_KB, wrow);
                    tma_load_2d(base + NA * TC_TILE_BYTES, mb, full_bar(stage), kb * TC_KB, sg.row0);
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) {
                // copies already issued may still be landing: give them time before teardown
                const uint64_t t0 = global_ns();
                while (global_ns() - t0 < 1000000ull) {
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (int item = blockIdx.x; ok && item < items; item += gridDim.x, ++it) {
                int grp, mt;
                Segment sg;
                decode(item, grp, mt, sg);
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(acce_bar(buf), acc_phase ^ 1u, abortp, args.status))
                    break;
                tc_fence_after();
                const int n_mma = max(16, (sg.n + 15) & ~15);
                const uint32_t idesc = umma_idesc_bf16(n_mma);
                const uint32_t d0 = tmem_base + (uint32_t)(buf * ACC_COLS);
                const int nkb = (args.K[grp] + TC_KB - 1) / TC_KB;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abortp, args.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t base = tiles + stage * STAGE_BYTES;
#pragma unroll
                    for (int k = 0; k < TC_KB / 16; ++k) {
                        const uint64_t bdesc = umma_desc_sw128(base + NA * TC_TILE_BYTES + k * 32);
                        const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
                        umma_bf16(d0, umma_desc_sw128(base + k * 32), bdesc, idesc, accum);
                        if (GATED)
                            umma_bf16(d0 + 128, umma_desc_sw128(base + TC_TILE_BYTES + k * 32), bdesc,
                                      idesc, accum);
                    }
                    umma_commit(empty_bar(stage));  // stage reusable once these MMAs are done
                    if (++stage == STAGES) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (ok)
                    umma_commit(accf_bar(buf));  // accumulator complete
            }
        }
    } else {
        // ---------------- epilogue (warps 2..5) ----------------
        const int quarter = warp & 3;  // TMEM lanes 32*quarter .. +31 belong to this warp
        int it = 0;
        for (int item = blockIdx.x; item < items; item += gridDim.x, ++it) {
            int grp, mt;
            Segment sg;
            decode(item, grp, mt, sg);
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            // every lane waits; the vote makes the decision uniform and reconverges the warp
            // for the warp-collective tcgen05.ld below
            const bool ready = mbar_wait(accf_bar(buf), acc_phase, abortp, args.status);
            if (!__all_sync(0xffffffffu, ready))
                break;
            tc_fence_after();
            const int rows = args.rows[grp];
            const int row = mt * TC_M + quarter * 32 + lane;  // output feature of this thread
            const int n = sg.n;
            __nv_bfloat16 *out = args.out[grp] + (size_t)sg.row0 * args.out_ld[grp] + row;
            const uint32_t t0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * ACC_COLS);
            for (int c0 = 0; c0 < n; c0 += 16) {
                uint32_t g[16], u[16];
                tmem_ld16(t0 + c0, g);
                if (GATED)
                    tmem_ld16(t0 + 128 + c0, u);
                tmem_ld_wait();
                if (row < rows) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (c0 + j < n) {
                            const float gv = __uint_as_float(g[j]);
                            const float res = GATED ? silu_f(gv) * __uint_as_float(u[j]) : gv;
                            out[(size_t)(c0 + j) * args.out_ld[grp]] = __float2bfloat16(res);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0)
                mbar_arrive(acce_bar(buf));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();  // lane 0 arrived from the issue loop: reconverge for the aligned dealloc
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"(TC_TMEM_COLS)
                     : "memory");
    }
}

// ---- gather of the token rows into sorted order (B operand of the gate/up pass) ---------

__global__ void __launch_bounds__(256)
gather_rows_kernel(const __nv_bfloat16 *__restrict__ x, const int32_t *__restrict__ perm, int A,
                   int H, int top_k, __nv_bfloat16 *__restrict__ x_sorted)
{
    const int vec_per_row = H >> 3;
    const size_t total = (size_t)A * vec_per_row;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const int r = (int)(i / vec_per_row);
        const int v = (int)(i - (size_t)r * vec_per_row);
        const int t = perm[r] / top_k;
        reinterpret_cast<uint4 *>(x_sorted + (size_t)r * H)[v] =
            reinterpret_cast<const uint4 *>(x + (size_t)t * H)[v];
    }
}

cudaError_t launch_gather_rows(const moe_config_t &c, const __nv_bfloat16 *x, const int32_t *perm,
                               int T, __nv_bfloat16 *x_sorted, cudaStream_t s)
{
    const int A = T * c.top_k;
    const size_t total = (size_t)A * (c.hidden >> 3);
    size_t blocks = (total + 255) / 256;
    const size_t cap = (size_t)sm_count() * 8;
    if (blocks > cap)
        blocks = cap;
    gather_rows_kernel<<<(unsigned)blocks, 256, 0, s>>>(x, perm, A, c.hidden, c.top_k, x_sorted);
    return cudaGetLastError();
}

// ---- host side: tensor maps and launches -------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// 2-D bf16 tensor [rows, cols] (cols contiguous), box = 64 columns x 128 rows, 128-byte swizzle.
static bool make_map(CUtensorMap *m, const void *base, uint64_t rows, uint64_t cols)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn)
        return false;
    if (base == nullptr || rows == 0 || cols == 0) {
        // group kind not present: a harmless 1-box map over a dummy extent is never used
        memset(m, 0, sizeof *m);
        return true;
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {TC_KB, TC_M};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool GATED>
static cudaError_t launch_tc(const TcArgs &a, const CUtensorMap (&maps)[6], cudaStream_t s)
{
    constexpr int STAGES = GATED ? TC_STAGES_GATED : TC_STAGES_DOWN;
    constexpr size_t SMEM = (size_t)STAGES * ((GATED ? 3 : 2) * TC_TILE_BYTES) + 1024;
    static bool configured[2] = {false, false};
    if (!configured[GATED]) {
        cudaError_t e = cudaFuncSetAttribute(ffn_tc_kernel<GATED>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM);
        if (e != cudaSuccess)
            return e;
        configured[GATED] = true;
    }
    ffn_tc_kernel<GATED><<<sm_count(), TC_THREADS, SMEM, s>>>(a, maps[0], maps[1], maps[2], maps[3],
                                                            maps[4], maps[5]);
    return cudaGetLastError();
}

cudaError_t launch_ffn_tc_gateup(const moe_config_t &c, const moe_weights_t &w,
                                 const __nv_bfloat16 *x, const __nv_bfloat16 *x_sorted, int T,
                                 PlanView plan, bool with_shared, __nv_bfloat16 *h,
                                 __nv_bfloat16 *h_shared, int32_t *status, cudaStream_t s)
{
    const uint64_t A = (uint64_t)T * c.top_k, H = c.hidden, E = c.n_experts;
    CUtensorMap maps[6];
    bool ok = make_map(&maps[0], w.w_gate, E * c.inter, H) && make_map(&maps[1], w.w_up, E * c.inter, H) &&
              make_map(&maps[2], x_sorted, A, H);
    if (with_shared)
        ok = ok && make_map(&maps[3], w.ws_gate, c.shared_inter, H) &&
             make_map(&maps[4], w.ws_up, c.shared_inter, H) && make_map(&maps[5], x, T, H);
    else
        ok = ok && make_map(&maps[3], nullptr, 0, 0) && make_map(&maps[4], nullptr, 0, 0) &&
             make_map(&maps[5], nullptr, 0, 0);
    if (!ok)
        return cudaErrorInvalidValue;
    TcArgs a{};
    a.rows[0] = c.inter;
    a.rows[1] = c.shared_inter;
    a.K[0] = a.K[1] = c.hidden;
    a.out[0] = h;
    a.out[1] = h_shared;
    a.out_ld[0] = c.inter;
    a.out_ld[1] = c.shared_inter;
    a.plan_header = plan.header;
    a.seg[0] = plan.tc_routed;
    a.seg[1] = plan.tc_shared;
    a.status = status;
    return launch_tc<true>(a, maps, s);
}

cudaError_t launch_ffn_tc_down(const moe_config_t &c, const moe_weights_t &w, int T, PlanView plan,
                               bool with_shared, const __nv_bfloat16 *h,
                               const __nv_bfloat16 *h_shared, __nv_bfloat16 *y,
                               __nv_bfloat16 *y_shared, int32_t *status, cudaStream_t s)
{
    const uint64_t A = (uint64_t)T * c.top_k, H = c.hidden, E = c.n_experts;
    CUtensorMap maps[6];
    bool ok = make_map(&maps[0], w.w_down, E * H, c.inter) && make_map(&maps[1], nullptr, 0, 0) &&
              make_map(&maps[2], h, A, c.inter) && make_map(&maps[4], nullptr, 0, 0);
    if (with_shared)
        ok = ok && make_map(&maps[3], w.ws_down, H, c.shared_inter) &&
             make_map(&maps[5], h_shared, T, c.shared_inter);
    else
        ok = ok && make_map(&maps[3], nullptr, 0, 0) && make_map(&maps[5], nullptr, 0, 0);
    if (!ok)
        return cudaErrorInvalidValue;
    TcArgs a{};
    a.rows[0] = a.rows[1] = c.hidden;
    a.K[0] = c.inter;
    a.K[1] = c.shared_inter;
    a.out[0] = y;
    a.out[1] = y_shared;
    a.out_ld[0] = a.out_ld[1] = c.hidden;
    a.plan_header = plan.header;
    a.seg[0] = plan.tc_routed;
    a.seg[1] = plan.tc_shared;
    a.status = status;
    return launch_tc<false>(a, maps, s);
}

}  // namespace moe

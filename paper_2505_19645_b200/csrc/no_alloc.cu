// moe_grouped_swiglu_static: the expert-FFN step for callers that cannot provide scratch.
//
// Some users of this library run where device allocation is off the table: a serving
// loop that fixed its memory plan at start-up and refuses any later cudaMalloc, a plugin
// inside a host framework that owns the allocator, a real-time path where an allocation
// could stall on a device-wide synchronisation.  For them the FFN step's scratch (segment
// plan + SwiGLU intermediates) lives in a fixed array inside the library image itself.
// The price: every GPU that loads the library carries MOE_STATIC_SCRATCH_BYTES until the
// process exits, sizes beyond it are refused, and all calls share (and overwrite) it.
#include <mutex>

#include "common.cuh"

namespace moe {

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// table, never a device address: the address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[MOE_STATIC_SCRATCH_BYTES];

static std::mutex g_scratch_mutex;
static void *g_scratch_addr[MAX_DEVICE_ORDINALS];  // per device ordinal, resolved on first use

// Device address of the scratch array on the CURRENT device (resolved once per device).
static moe_status_t static_scratch_address(char **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (dev < 0 || dev >= MAX_DEVICE_ORDINALS)
        return MOE_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p)
            return MOE_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = static_cast<char *>(g_scratch_addr[dev]);
    return MOE_OK;
}

// Only the regions the FFN step touches, packed from offset 0.
static Workspace static_scratch_layout(const moe_config_t &c, int T)
{
    Workspace w{};
    const size_t A = (size_t)T * c.top_k;
    WorkspaceCarver cut(w);
    w.status = cut.take(64 * 4);
    w.plan_header = cut.take(PLAN_HEADER_INTS * 4);
    w.plan_seg = cut.take(sizeof(Segment) * (size_t)max_segments(c.n_experts, (int)A));
    w.plan_pairs = cut.take(sizeof(PairEntry) * (size_t)max_segments(c.n_experts, (int)A));
    w.plan_done = cut.take(4 * ((size_t)max_segments(c.n_experts, (int)A) + max_shared_segments(T)));
    w.plan_done_shared_at = (size_t)max_segments(c.n_experts, (int)A);
    w.x_sorted = cut.take(A * (size_t)c.hidden * 2);
    w.h = cut.take(A * (size_t)c.inter * 2);
    w.h_shared = cut.take((size_t)T * c.shared_inter * 2);
    w.total = cut.off;
    return w;
}

}  // namespace moe

using namespace moe;

extern "C" {

moe_status_t moe_grouped_swiglu_static(const moe_config_t *cfg, const moe_weights_t *w,
                                       const void *x, int32_t T, const int32_t *offsets,
                                       const int32_t *perm, const int32_t *active,
                                       const int32_t *n_active, void *y, void *shared_y,
                                       void *stream)
{
    moe_status_t st = check_config(cfg);
    if (st != MOE_OK)
        return st;
    if ((st = check_tokens(cfg, T)) != MOE_OK)
        return st;
    if (!weights_ok(cfg, w, false, true) || !x || !offsets || !perm || !active || !n_active || !y)
        return MOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y) || (shared_y && !aligned16(shared_y)))
        return MOE_ERR_INVALID_ARG;
    const Workspace L = static_scratch_layout(*cfg, T);
    if (L.total > (size_t)MOE_STATIC_SCRATCH_BYTES)
        return MOE_ERR_WORKSPACE;  // request does not fit the built-in scratch
    if ((st = check_device()) != MOE_OK)
        return st;
    char *scratch = nullptr;
    if ((st = static_scratch_address(&scratch)) != MOE_OK)
        return st;
    int launches = 0;
    // The plan kernel, first in the sequence, clears the progress counters and rewrites the
    // whole plan; the down pass reads a segment of h only once the gate/up pass has counted
    // it complete.  Nothing else in the array has to start at zero (the status word is
    // zero when the library is loaded and is cleared by moe_check_static after a report).
    return run_ffn(*cfg, *w, static_cast<const __nv_bfloat16 *>(x), T, offsets, perm,
                   static_cast<__nv_bfloat16 *>(y), static_cast<__nv_bfloat16 *>(shared_y), scratch,
                   L, static_cast<cudaStream_t>(stream), launches);
}

moe_status_t moe_check_static(void *stream)
{
    moe_status_t st = check_device();
    if (st != MOE_OK)
        return st;
    char *scratch = nullptr;
    if ((st = static_scratch_address(&scratch)) != MOE_OK)
        return st;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return MOE_ERR_CUDA;
    // the status region is the first of the array (static_scratch_layout)
    return read_and_clear_status(scratch);
}

moe_status_t moe_selftest_wait_limit_static(int32_t limit_us, void *stream)
{
    if (limit_us < 1 || limit_us > 1000000)
        return MOE_ERR_INVALID_ARG;
    moe_status_t st = check_device();
    if (st != MOE_OK)
        return st;
    char *scratch = nullptr;
    if ((st = static_scratch_address(&scratch)) != MOE_OK)
        return st;
    int32_t *status = reinterpret_cast<int32_t *>(scratch);
    if (launch_wait_limit_selftest(status, status + 2, limit_us, static_cast<cudaStream_t>(stream)) !=
        cudaSuccess)
        return MOE_ERR_CUDA;
    return MOE_OK;
}

}  // extern "C"

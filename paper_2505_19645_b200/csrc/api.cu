// C ABI: argument validation, workspace carving and launch sequencing.  No compute here.
#include <stdlib.h>

#include <mutex>

#include "common.cuh"

namespace moe {

int sm_count()
{
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64)
        return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

void prefer_max_shared_carveout(const void *kernel)
{
    // a handful of kernels: a small table of those already configured (a race between two
    // threads at worst sets the attribute twice)
    struct Key {
        const void *kernel;
        int device;
    };
    static Key seen[256];
    static int n_seen = 0;
    int dev = 0;
    cudaGetDevice(&dev);
    for (int i = 0; i < n_seen; ++i)
        if (seen[i].kernel == kernel && seen[i].device == dev)
            return;
    cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                         cudaSharedmemCarveoutMaxShared);
    if (n_seen < 256)
        seen[n_seen++] = Key{kernel, dev};
}

// MOE_NO_PDL=1 in the environment launches every kernel with plain stream ordering.
bool pdl_enabled()
{
    static const bool on = [] {
        const char *e = getenv("MOE_NO_PDL");
        return !(e && e[0] == '1');
    }();
    return on;
}

int schedule_override()
{
    static const int v = [] {
        const char *e = getenv("MOE_FF_RR");
        return !e ? -1 : (e[0] == '1' ? 1 : (e[0] == '0' ? 0 : -1));
    }();
    return v;
}

int geometry_override()
{
    static const int v = [] {
        const char *e = getenv("MOE_FF_WIDE");
        return !e ? -1 : (e[0] == '1' ? 1 : (e[0] == '0' ? 0 : -1));
    }();
    return v;
}

static thread_local int g_last_launches = 0;

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

moe_status_t check_config(const moe_config_t *c)
{
    if (!c)
        return MOE_ERR_INVALID_ARG;
    if (c->hidden < 32 || c->hidden % 32 || c->inter < 32 || c->inter % 32)
        return MOE_ERR_INVALID_ARG;
    if (c->shared_inter < 0 || c->shared_inter % 32)
        return MOE_ERR_INVALID_ARG;
    if (c->n_experts < 1 || c->n_experts > MOE_MAX_EXPERTS)
        return MOE_ERR_INVALID_ARG;
    if (c->top_k < 1 || c->top_k > MOE_MAX_TOPK || c->top_k > c->n_experts)
        return MOE_ERR_INVALID_ARG;
    if (c->score_fn != MOE_SCORE_SOFTMAX && c->score_fn != MOE_SCORE_SIGMOID)
        return MOE_ERR_INVALID_ARG;
    return MOE_OK;
}

moe_status_t check_tokens(const moe_config_t *c, int64_t T)
{
    if (T < 1 || T * c->top_k >= (1 << 24))
        return MOE_ERR_INVALID_ARG;
    return MOE_OK;
}

// The kernels are built for sm_100a only.
moe_status_t check_device()
{
    static int ok[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (dev < 0 || dev >= 64)
        return MOE_ERR_UNSUPPORTED;
    if (ok[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
            return MOE_ERR_CUDA;
        ok[dev] = major == 10 ? 1 : -1;
    }
    return ok[dev] == 1 ? MOE_OK : MOE_ERR_UNSUPPORTED;
}

bool weights_ok(const moe_config_t *c, const moe_weights_t *w, bool need_router,
                       bool need_experts)
{
    if (!w)
        return false;
    if (need_router) {
        if (!w->w_router || !aligned16(w->w_router))
            return false;
        if (c->shared_inter > 0 && c->shared_gate && (!w->w_shared_gate || !aligned16(w->w_shared_gate)))
            return false;
    }
    if (need_experts) {
        if (!w->w_gate || !w->w_up || !w->w_down)
            return false;
        if (!aligned16(w->w_gate) || !aligned16(w->w_up) || !aligned16(w->w_down))
            return false;
        if (c->shared_inter > 0) {
            if (!w->ws_gate || !w->ws_up || !w->ws_down)
                return false;
            if (!aligned16(w->ws_gate) || !aligned16(w->ws_up) || !aligned16(w->ws_down))
                return false;
        }
    }
    return true;
}

#define MOE_TRY_LAUNCH(expr)            \
    do {                                \
        if ((expr) != cudaSuccess)      \
            return MOE_ERR_CUDA;        \
        ++launches;                     \
    } while (0)

// Optional event pair around one stage of moe_verify_layer (see moe_profile_stage).
struct StageProbe {
    int stage = -1;
    cudaEvent_t start = nullptr, stop = nullptr;
};
static thread_local StageProbe g_probe;
static thread_local bool g_probe_armed = false;  // only moe_verify_layer arms it

#define MOE_STAGE(stage_id, expr)                                             \
    do {                                                                      \
        const bool probe_ = g_probe_armed && g_probe.stage == (stage_id);     \
        if (probe_ && cudaEventRecord(g_probe.start, s) != cudaSuccess)       \
            return MOE_ERR_CUDA;                                              \
        MOE_TRY_LAUNCH(expr);                                                 \
        if (probe_ && cudaEventRecord(g_probe.stop, s) != cudaSuccess)        \
            return MOE_ERR_CUDA;                                              \
    } while (0)

// The stream must be idle.  A raised word is reported once: it is cleared after it has been read.
moe_status_t read_and_clear_status(void *status_region)
{
    int32_t word[2] = {0, 0};
    if (cudaMemcpy(word, status_region, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (word[1] != STATUS_MAGIC || word[0] == 0)
        return MOE_OK;  // never initialised: no call has run on this workspace yet
    if (cudaMemset(status_region, 0, sizeof(int32_t)) != cudaSuccess)
        return MOE_ERR_CUDA;
    return MOE_ERR_TIMEOUT;
}

PlanView plan_view(char *ws, const Workspace &L, int seg_rows)
{
    return PlanView{seg_rows, reinterpret_cast<int32_t *>(ws + L.plan_header),
                    reinterpret_cast<Segment *>(ws + L.plan_seg),
                    reinterpret_cast<PairEntry *>(ws + L.plan_pairs),
                    reinterpret_cast<int32_t *>(ws + L.plan_done),
                    reinterpret_cast<int32_t *>(ws + L.plan_done) + L.plan_done_shared_at};
}

moe_status_t run_ffn(const moe_config_t &c, const moe_weights_t &w, const __nv_bfloat16 *x, int T,
                     const int32_t *offsets, const int32_t *perm, __nv_bfloat16 *y,
                     __nv_bfloat16 *shared_y, char *ws, const Workspace &L, cudaStream_t s,
                     int &launches, bool plan_ready, int shared_parts, int routed_parts,
                     bool gathered)
{
    const bool with_shared = shared_y != nullptr && c.shared_inter > 0;
    const PlanView plan = plan_view(ws, L, ffn_segment_rows(c, T));
    int32_t *status = reinterpret_cast<int32_t *>(ws + L.status);
    __nv_bfloat16 *h = reinterpret_cast<__nv_bfloat16 *>(ws + L.h);
    __nv_bfloat16 *hs = reinterpret_cast<__nv_bfloat16 *>(ws + L.h_shared);
    __nv_bfloat16 *xs = reinterpret_cast<__nv_bfloat16 *>(ws + L.x_sorted);
    if (!plan_ready)
        MOE_STAGE(MOE_STAGE_PLAN, launch_plan(c, T, offsets, status, plan, s));
    if (!gathered)
        MOE_STAGE(MOE_STAGE_GATHER, launch_gather_rows(c, x, perm, T, xs, s));
    MOE_STAGE(MOE_STAGE_GATE_UP,
              launch_ffn_gateup(c, w, x, xs, T, plan, with_shared, h, hs, status, s));
    MOE_STAGE(MOE_STAGE_DOWN,
              launch_ffn_down(c, w, T, plan, with_shared, h, hs, y, shared_y, shared_parts,
                              routed_parts, status, s));
    return MOE_OK;
}

}  // namespace moe

using namespace moe;

// Copies of the layer's intermediates for the caller (moe_debug_out_t), enqueued behind the layer.
static moe_status_t copy_debug_out(const moe_config_t &c, int T, const moe_debug_out_t *dbg,
                                   const char *base, const Workspace &L, cudaStream_t s)
{
    if (!dbg)
        return MOE_OK;
    const size_t A = (size_t)T * c.top_k, E = c.n_experts;
    struct Copy {
        void *dst;
        size_t src;
        size_t bytes;
    } copies[] = {
        {dbg->logits, L.logits, (size_t)T * E * 4}, {dbg->topk_idx, L.topk_idx, A * 4},
        {dbg->topk_w, L.topk_w, A * 4},             {dbg->counts, L.counts, E * 4},
        {dbg->offsets, L.offsets, (E + 1) * 4},     {dbg->perm, L.perm, A * 4},
        {dbg->inv_perm, L.inv_perm, A * 4},         {dbg->active, L.active, E * 4},
        {dbg->n_active, L.n_active, 4},
    };
    for (const Copy &cp : copies)
        if (cp.dst && cudaMemcpyAsync(cp.dst, base + cp.src, cp.bytes, cudaMemcpyDeviceToDevice, s) !=
                          cudaSuccess)
            return MOE_ERR_CUDA;
    return MOE_OK;
}

extern "C" {

size_t moe_workspace_bytes(const moe_config_t *cfg, int32_t max_tokens)
{
    if (check_config(cfg) != MOE_OK || check_tokens(cfg, max_tokens) != MOE_OK)
        return 0;
    return workspace_layout(*cfg, max_tokens).total;
}

moe_status_t moe_router_logits(const moe_config_t *cfg, const moe_weights_t *w, const void *x,
                               int32_t T, float *logits, float *shared_scale, void *stream)
{
    moe_status_t st = check_config(cfg);
    if (st != MOE_OK)
        return st;
    if ((st = check_tokens(cfg, T)) != MOE_OK)
        return st;
    if (!weights_ok(cfg, w, true, false) || !x || !logits || !aligned16(x) || !aligned16(logits))
        return MOE_ERR_INVALID_ARG;
    if ((st = check_device()) != MOE_OK)
        return st;
    int launches = 0;
    MOE_TRY_LAUNCH(launch_router_logits(*cfg, *w, static_cast<const __nv_bfloat16 *>(x), T, logits,
                                        shared_scale, static_cast<cudaStream_t>(stream)));
    return MOE_OK;
}

moe_status_t moe_route_topk(const moe_config_t *cfg, const float *logits, int32_t T,
                            int32_t *topk_idx, float *topk_w, void *stream)
{
    moe_status_t st = check_config(cfg);
    if (st != MOE_OK)
        return st;
    if ((st = check_tokens(cfg, T)) != MOE_OK)
        return st;
    if (!logits || !topk_idx || !topk_w || !aligned16(logits) || !aligned16(topk_idx) ||
        !aligned16(topk_w))
        return MOE_ERR_INVALID_ARG;
    if ((st = check_device()) != MOE_OK)
        return st;
    int launches = 0;
    MOE_TRY_LAUNCH(launch_route_topk(*cfg, logits, T, topk_idx, topk_w,
                                     static_cast<cudaStream_t>(stream)));
    return MOE_OK;
}

moe_status_t moe_permute(const moe_config_t *cfg, const int32_t *topk_idx, int32_t T,
                         int32_t *counts, int32_t *offsets, int32_t *perm, int32_t *inv_perm,
                         int32_t *active, int32_t *n_active, void *stream)
{
    moe_status_t st = check_config(cfg);
    if (st != MOE_OK)
        return st;
    if ((st = check_tokens(cfg, T)) != MOE_OK)
        return st;
    if (!topk_idx || !counts || !offsets || !perm || !inv_perm || !active || !n_active)
        return MOE_ERR_INVALID_ARG;
    if (!aligned16(topk_idx) || !aligned16(perm) || !aligned16(inv_perm))
        return MOE_ERR_INVALID_ARG;
    if ((st = check_device()) != MOE_OK)
        return st;
    int launches = 0;
    MOE_TRY_LAUNCH(launch_permute(*cfg, topk_idx, T, counts, offsets, perm, inv_perm, active,
                                  n_active, static_cast<cudaStream_t>(stream)));
    return MOE_OK;
}

moe_status_t moe_grouped_swiglu(const moe_config_t *cfg, const moe_weights_t *w, const void *x,
                                int32_t T, const int32_t *offsets, const int32_t *perm,
                                const int32_t *active, const int32_t *n_active, void *y,
                                void *shared_y, void *ws, size_t ws_bytes, void *stream)
{
    moe_status_t st = check_config(cfg);
    if (st != MOE_OK)
        return st;
    if ((st = check_tokens(cfg, T)) != MOE_OK)
        return st;
    if (!weights_ok(cfg, w, false, true) || !x || !offsets || !perm || !active || !n_active || !y ||
        !ws)
        return MOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y) || !aligned16(ws) || (shared_y && !aligned16(shared_y)))
        return MOE_ERR_INVALID_ARG;
    const Workspace L = workspace_layout(*cfg, T);
    if (ws_bytes < L.total)
        return MOE_ERR_WORKSPACE;
    if ((st = check_device()) != MOE_OK)
        return st;
    int launches = 0;
    return run_ffn(*cfg, *w, static_cast<const __nv_bfloat16 *>(x), T, offsets, perm,
                   static_cast<__nv_bfloat16 *>(y), static_cast<__nv_bfloat16 *>(shared_y),
                   static_cast<char *>(ws), L, static_cast<cudaStream_t>(stream), launches);
}

moe_status_t moe_combine(const moe_config_t *cfg, const void *y, const int32_t *inv_perm,
                         const float *topk_w, const void *shared_y, const float *shared_scale,
                         int32_t T, void *out, void *stream)
{
    moe_status_t st = check_config(cfg);
    if (st != MOE_OK)
        return st;
    if ((st = check_tokens(cfg, T)) != MOE_OK)
        return st;
    if (!y || !inv_perm || !topk_w || !out || !aligned16(y) || !aligned16(out) ||
        (shared_y && !aligned16(shared_y)))
        return MOE_ERR_INVALID_ARG;
    if ((st = check_device()) != MOE_OK)
        return st;
    int launches = 0;
    MOE_TRY_LAUNCH(launch_combine(*cfg, static_cast<const __nv_bfloat16 *>(y), 1, inv_perm, topk_w,
                                  static_cast<const __nv_bfloat16 *>(shared_y), 1, shared_scale, T,
                                  static_cast<__nv_bfloat16 *>(out),
                                  static_cast<cudaStream_t>(stream)));
    return MOE_OK;
}

moe_status_t moe_verify_layer(const moe_config_t *cfg, const moe_weights_t *w, const void *x,
                              int32_t B, int32_t gamma, void *out, const moe_debug_out_t *dbg,
                              void *ws, size_t ws_bytes, void *stream)
{
    g_last_launches = 0;
    moe_status_t st = check_config(cfg);
    if (st != MOE_OK)
        return st;
    if (B < 1 || gamma < 0)
        return MOE_ERR_INVALID_ARG;
    const int64_t T64 = (int64_t)B * ((int64_t)gamma + 1);
    if ((st = check_tokens(cfg, T64)) != MOE_OK)
        return st;
    const int T = (int)T64;
    if (!weights_ok(cfg, w, true, true) || !x || !out || !ws || !aligned16(x) || !aligned16(out) ||
        !aligned16(ws))
        return MOE_ERR_INVALID_ARG;
    const Workspace L = workspace_layout(*cfg, T);
    if (ws_bytes < L.total)
        return MOE_ERR_WORKSPACE;
    if ((st = check_device()) != MOE_OK)
        return st;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char *base = static_cast<char *>(ws);
    const __nv_bfloat16 *xb = static_cast<const __nv_bfloat16 *>(x);
    if (layer_small_applies(*cfg, T)) {
        // a handful of tokens: the whole layer is one launch (its time is recorded as the
        // gate/up stage's, the stage that dominates it)
        const bool probe_ = g_probe.stage == MOE_STAGE_GATE_UP;
        if (probe_ && cudaEventRecord(g_probe.start, s) != cudaSuccess)
            return MOE_ERR_CUDA;
        const cudaError_t err =
            launch_layer_small(*cfg, *w, xb, T, static_cast<__nv_bfloat16 *>(out), base, L, s);
        if (err == cudaSuccess) {
            if (probe_ && cudaEventRecord(g_probe.stop, s) != cudaSuccess)
                return MOE_ERR_CUDA;
            g_last_launches = 1;
            return copy_debug_out(*cfg, T, dbg, base, L, s);
        }
        // a context that cannot hold one CTA per SM at once (SMs set aside for others) refuses
        // the cooperative launch: nothing was enqueued, the kernel sequence below serves the call
        if (err != cudaErrorCooperativeLaunchTooLarge)
            return MOE_ERR_CUDA;
        (void)cudaGetLastError();
    }
    float *logits = reinterpret_cast<float *>(base + L.logits);
    int32_t *topk_idx = reinterpret_cast<int32_t *>(base + L.topk_idx);
    float *topk_w = reinterpret_cast<float *>(base + L.topk_w);
    float *shared_scale = reinterpret_cast<float *>(base + L.shared_scale);
    int32_t *counts = reinterpret_cast<int32_t *>(base + L.counts);
    int32_t *offsets = reinterpret_cast<int32_t *>(base + L.offsets);
    int32_t *active = reinterpret_cast<int32_t *>(base + L.active);
    int32_t *n_active = reinterpret_cast<int32_t *>(base + L.n_active);
    int32_t *perm = reinterpret_cast<int32_t *>(base + L.perm);
    int32_t *inv_perm = reinterpret_cast<int32_t *>(base + L.inv_perm);
    __nv_bfloat16 *y = reinterpret_cast<__nv_bfloat16 *>(base + L.y);
    const bool has_shared = cfg->shared_inter > 0;
    const bool gated = has_shared && cfg->shared_gate;
    __nv_bfloat16 *ys = has_shared ? reinterpret_cast<__nv_bfloat16 *>(base + L.y_shared) : nullptr;

    int launches = 0;
    struct Arm {
        Arm() { g_probe_armed = true; }
        ~Arm() { g_probe_armed = false; }
    } arm;
    const PlanView plan = plan_view(base, L, ffn_segment_rows(*cfg, T));
    int32_t *status = reinterpret_cast<int32_t *>(base + L.status);
    int logit_chunks = 0;  // > 0: the logits are still partial sums per k chunk (summed by the top-k)
    if (router_logits_tc_applies(*cfg, T)) {
        const bool probe_ = g_probe_armed && g_probe.stage == MOE_STAGE_ROUTER_LOGITS;
        if (probe_ && cudaEventRecord(g_probe.start, s) != cudaSuccess)
            return MOE_ERR_CUDA;
        if (launch_router_logits_tc(*cfg, *w, xb, T,
                                    reinterpret_cast<__nv_bfloat16 *>(base + L.rl_planes),
                                    reinterpret_cast<float *>(base + L.rl_partial), s,
                                    plan.done_shared, max_shared_segments(T), status,
                                    &launches, &logit_chunks) != cudaSuccess)
            return MOE_ERR_CUDA;
        if (probe_ && cudaEventRecord(g_probe.stop, s) != cudaSuccess)
            return MOE_ERR_CUDA;
    } else {
        MOE_STAGE(MOE_STAGE_ROUTER_LOGITS,
                  launch_router_logits(*cfg, *w, xb, T, logits, gated ? shared_scale : nullptr, s,
                                       plan.done_shared, max_shared_segments(T), status));
    }
    // the grouping kernel also writes the FFN segment plan (one launch fewer); for a small
    // batch it selects the experts and gathers the token rows as well (three fewer)
    const bool small = route_group_small_applies(*cfg, T);
    if (small) {
        MOE_STAGE(MOE_STAGE_PERMUTE,
                  launch_route_group_small(*cfg, logits, xb, T, topk_idx, topk_w, counts, offsets,
                                           perm, inv_perm, active, n_active, status, plan,
                                           reinterpret_cast<__nv_bfloat16 *>(base + L.x_sorted), s));
    } else {
        if (logit_chunks > 0)
            MOE_STAGE(MOE_STAGE_ROUTE_TOPK,
                      launch_route_topk_sum(*cfg, reinterpret_cast<const float *>(base + L.rl_partial),
                                            logit_chunks, cfg->n_experts + (gated ? 1 : 0),
                                            w->router_bias, T, logits, gated ? shared_scale : nullptr,
                                            topk_idx, topk_w, s));
        else
            MOE_STAGE(MOE_STAGE_ROUTE_TOPK, launch_route_topk(*cfg, logits, T, topk_idx, topk_w, s));
        MOE_STAGE(MOE_STAGE_PERMUTE,
                  launch_permute(*cfg, topk_idx, T, counts, offsets, perm, inv_perm, active,
                                 n_active, s, &plan, status));
    }
    const int shared_parts = has_shared ? shared_down_parts(*cfg) : 1;
    const int routed_parts = routed_down_parts(*cfg, T);
    st = run_ffn(*cfg, *w, xb, T, offsets, perm, y, ys, base, L, s, launches, true, shared_parts,
                 routed_parts, small);
    if (st != MOE_OK)
        return st;
    MOE_STAGE(MOE_STAGE_COMBINE,
              launch_combine(*cfg, y, routed_parts, inv_perm, topk_w, ys, shared_parts, gated ? shared_scale : nullptr, T,
                             static_cast<__nv_bfloat16 *>(out), s));
    g_last_launches = launches;

    return copy_debug_out(*cfg, T, dbg, base, L, s);
}

moe_status_t moe_check(void *ws, void *stream)
{
    if (!ws)
        return MOE_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return MOE_ERR_CUDA;
    return read_and_clear_status(ws);
}

moe_status_t moe_workspace_region(const moe_config_t *cfg, int32_t T, int32_t index, size_t *offset,
                                  size_t *bytes)
{
    if (check_config(cfg) != MOE_OK || check_tokens(cfg, T) != MOE_OK || !offset || !bytes)
        return MOE_ERR_INVALID_ARG;
    const Workspace L = workspace_layout(*cfg, T);
    if (index < 0 || index >= L.n_regions)
        return MOE_ERR_INVALID_ARG;
    *offset = L.region_off[index];
    *bytes = L.region_bytes[index];
    return MOE_OK;
}

moe_status_t moe_selftest_wait_limit(void *ws, int32_t limit_us, void *stream)
{
    if (!ws || !aligned16(ws) || limit_us < 1 || limit_us > 1000000)
        return MOE_ERR_INVALID_ARG;
    moe_status_t st = check_device();
    if (st != MOE_OK)
        return st;
    int32_t *status = static_cast<int32_t *>(ws);  // the status region is the first of the workspace
    int launches = 0;
    MOE_TRY_LAUNCH(launch_wait_limit_selftest(status, status + 2, limit_us,
                                              static_cast<cudaStream_t>(stream)));
    MOE_TRY_LAUNCH(launch_tagged_wait_selftest(status, limit_us, static_cast<cudaStream_t>(stream)));
    return MOE_OK;
}

moe_status_t moe_profile_stage(int32_t stage, void *start_event, void *stop_event)
{
    if (stage > MOE_STAGE_GATHER || (stage >= 0 && (!start_event || !stop_event)))
        return MOE_ERR_INVALID_ARG;
    g_probe.stage = stage < 0 ? -1 : stage;
    g_probe.start = static_cast<cudaEvent_t>(start_event);
    g_probe.stop = static_cast<cudaEvent_t>(stop_event);
    return MOE_OK;
}

int32_t moe_last_launch_count(void) { return g_last_launches; }

const char *moe_status_string(moe_status_t s)
{
    switch (s) {
    case MOE_OK: return "ok";
    case MOE_ERR_INVALID_ARG: return "invalid argument";
    case MOE_ERR_UNSUPPORTED: return "unsupported (needs an sm_100a GPU)";
    case MOE_ERR_WORKSPACE: return "workspace too small";
    case MOE_ERR_CUDA: return "CUDA runtime error";
    case MOE_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

}  // extern "C"

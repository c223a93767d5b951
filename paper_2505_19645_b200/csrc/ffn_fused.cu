// Expert FFN (gate/up + SwiGLU, and down projection) for every group size: the activated
// experts' weights are streamed from HBM exactly once by TMA through a ring of shared-memory
// slots and contracted on the tensor cores (tcgen05.mma, fp32 accumulators in TMEM).
//
// Orientation.  Measured on this part, one tcgen05.mma kind::f16 of shape M x N x 16 occupies
// the tensor pipe for max(48.5, N / 2) cycles, whatever M in {64, 128} is and whether or not
// consecutive instructions share an accumulator.  The weight rows are therefore the M operand
// (blocks of 128 rows: a gate block and the matching up block, or two blocks of W_down) and the
// group's token rows are the N operand (a segment of up to 128 or 256 rows, rounded up to 16):
// the instruction time follows the number of tokens, so a group of 160 rows costs 160/256 of a
// full tile instead of two full instructions, and a handful of tokens cost the 48.5-cycle floor
// -- 8 KB of weights per 97 cycles, far more than HBM delivers per SM in that time.  The kernel
// stays bandwidth-bound from one token per expert up to the roofline ridge (Sec. 3.3: the
// layer's time is the time to load the activated experts), and full 256-token segments run the
// instruction at its full rate.  In TMEM a lane is a weight row (an output feature) and a
// column a token: an epilogue thread owns one feature and walks the tokens.
//
// Work partition.  Output features are independent, so the weight rows of all routed
// groups are laid end to end (one position = 16 rows of one group for one of its segments)
// and the CTAs of the persistent grid claim chunks of positions at run time from a grid-wide
// counter (chunk ends on tile boundaries, sizes shrinking as the work runs out), or, where
// chunks would be too short or too many, single (segment, tile, k chunk) items: a CTA that
// starts late or runs slowly takes less, there is no tile-count quantisation and no tail wave.
// The shared expert's rows are cut into (tile, k chunk, segment) units that are dealt
// round-robin to the CTAs; they depend on nothing the layer computes, so they run before the
// routing result exists.  Tiles have at most 128 features (gate/up: two blocks, gate and up)
// or 256 (down: two blocks).  The units of one shared tile run at the same time on
// neighbouring CTAs and meet in L2.
//
// Between the passes.  The gate/up pass counts, per segment, the 16-column units of h its
// epilogue warps have stored (a releasing reduction); the down pass starts while the gate/up
// pass is still running and fetches a segment's rows of h once the segment's count is
// complete (acquire load, then a proxy fence before the TMA loads).
//
// Two ring geometries, chosen by the host per call.  Streaming (segments of up to 128 rows): a
// weight slot holds two 64-element k boxes of one tile (64 KB for a full tile), so that one
// producer/consumer hand-shake moves enough bytes to keep HBM busy and every weight row is
// requested in 256 contiguous bytes; two sets of accumulators, so the epilogue of one tile
// runs under the instructions of the next.  Contraction (segments of up to 256 rows, for
// groups in the hundreds of rows): one k box per slot (32 KB) and per token entry (up to
// 32 KB), four weight slots and three token entries, one set of accumulators of 2 x 256
// columns.  The token operand lives in a second ring whose entries are sized by the
// segment's row count and never wrap.
//
// CTA = 11 warps.  warp 0: weight producer (one lane issues TMA), warp 1: MMA issuer (one
// lane) and owner of the TMEM allocation, warp 2: token-operand producer, warps 3..10:
// epilogue, two warps per TMEM lane quarter that take alternate 16-token chunks (tcgen05.ld,
// SwiGLU, transposition, 16-byte bf16 stores): where no second set of accumulators exists the
// epilogue is not hidden behind the next tile, and two warps per scheduler hide its latencies.  Rings and the
// accumulator sets are handed over through mbarriers.  Every wait is bounded: when one
// gives up it raises the CTA's abort flag and the device status word, all roles leave their
// loops, TMEM is freed and the kernel returns.
//
// Programmatic dependent launch: the kernels may start while their predecessor in the stream
// is still running.  Work that depends only on the caller's inputs (shared-expert tiles in the
// gate/up pass, weight prefetch in the down pass) is done before griddepcontrol.wait, so it
// overlaps the routing kernels; everything produced inside the layer is touched after it,
// except h, which the down pass takes segment by segment as described above.
#include <math.h>
#include <string.h>

#include <mutex>

#include "tc_ptx.cuh"

namespace moe {

constexpr int FF_EPI_WARPS = 8;
constexpr int FF_THREADS = 32 * (3 + FF_EPI_WARPS);
constexpr int FF_MAX_W_SLOTS = 8;
constexpr int FF_X_ENTRIES = 8;                               // token-ring entries in flight
constexpr int FF_SEG = SEG_TOKENS;        // token rows per segment in the streaming geometry
constexpr int FF_SEG_WIDE = 2 * SEG_TOKENS;  // ... in the contraction geometry (the MMA's N limit)
constexpr int FF_TMEM_COLS = 512;
constexpr int FF_SMEM_LIMIT = 227 * 1024;
constexpr int FF_X_UNIT = 2048;  // token ring unit: 16 rows x 128 bytes
constexpr int FF_HEIGHTS = 4;    // TMA box heights for weight tiles: 128, 64, 32, 16 rows

struct FfnArgs {
    int rows[2];   // output features per group kind (0 routed, 1 shared), multiples of 16
    int K[2];      // reduction length per group kind
    __nv_bfloat16 *out[2];
    int out_ld[2];
    const int32_t *plan_header;  // [0] = [1] = number of segments
    const Segment *seg;
    const PairEntry *pairs;      // one entry per segment, with its group
    int32_t *claim_counter;      // grid-wide: next unclaimed routed position / item of this pass
    int32_t *done[2];            // per segment of each group kind: 16-column units of h finished
                                 // by the gate/up pass, summed over its four epilogue warps
    int round_robin;             // routed work dealt as (pair, tile) items instead of ranges
    int32_t *status;
    int T;             // token rows (the shared expert's group)
    int with_shared;   // shared expert present in this launch
    int shared_ksplit;   // k chunks of the shared expert's reduction (down pass; 1 = whole K):
                         // chunk s covers [s * shared_kchunk, ...) and writes its partial sums
                         // to out[1] + s * shared_part_stride
    int shared_kchunk;   // multiple of 128
    long long shared_part_stride;  // elements
    int routed_ksplit;   // the same for the routed groups (round-robin mode of the down pass only)
    int routed_kchunk;
    long long routed_part_stride;
    int shared_tiles;  // tiles of the shared expert's rows; (tile, k chunk, segment) units are dealt
                       // round-robin to the CTAs; the first (units % tiles) tiles have one
                       // 16-row unit more
    int max_tile;      // weight rows per tile: 128 (gate + up stacked) or 256 (down)
    int kboxes;        // 64-element k boxes per weight slot
    int w_slot_bytes;  // capacity of a weight slot
    int n_w_slots;
    int x_units;       // token ring size in FF_X_UNIT units
    int wait_us;       // limit of every wait inside the kernel, microseconds
    int seg_rows;      // token rows per segment of the routed groups (as in the plan): 128 or 256
    int shared_seg;    // token rows per segment of the shared expert: seg_rows, or 64 for
                       // 64 < T <= 128 with the small token ring (no entry beyond 16 KB)
    int acc_sets;      // accumulator sets in TMEM: 2 (segments up to 128 rows: a set is 2 x 128
                       // columns) or 1 (up to 256 rows: 2 x 256 columns)
};

// Tensor maps of one pass: weights [kind][matrix][box height], token operand [kind][box height].
struct FfnMaps {
    CUtensorMap w[2][2][FF_HEIGHTS];
    CUtensorMap x[2][FF_HEIGHTS];
};

// ---- kernel ----------------------------------------------------------------------------

// One work item: one segment of token rows of a group against one tile of its weight rows.
struct Item {
    int grp;     // 0 routed, 1 shared
    int expert;  // routed expert id (0 for the shared expert)
    int f0;      // first output feature (weight row inside the expert), multiple of 16
    int h;       // output features of the tile, multiple of 16
    int row0;    // first token row (sorted row for routed groups, token for the shared expert)
    int n;       // token rows, 1..seg_rows
    int seg;     // index of the segment's progress counter (plan index; shared: segment number)
    int w_once;  // the tile's weights are read by this item only
    int k0, k1;  // reduction range [k0, k1)
    long long out_off;  // element offset of this item's output plane (k chunk) in out[grp]
};

// Hand-over of the routed work a CTA claims at run time.  One thread of the CTA (the weight
// producer) claims chunks from a grid-wide counter and publishes them in a small ring; the
// other roles read the same sequence, so all roles walk identical items.
constexpr int FF_CLAIMS = 4;      // ring entries
constexpr int FF_CLAIM_READERS = 2 + FF_EPI_WARPS;  // token producer, MMA issuer, epilogue warps

constexpr int FF_CLAIM_WORDS = 8;  // lo, hi, and (round-robin mode) the item's group, decoded
struct ClaimRing {
    int *data;                 // shared memory [FF_CLAIMS][FF_CLAIM_WORDS]
    uint32_t full0, empty0;    // shared addresses of the barrier arrays [FF_CLAIMS]
    volatile int *abort_flag;
    int32_t *status;
};

// Walks the items of one CTA: its units of the shared expert first (dealt round-robin: they
// depend on nothing the layer computes), then chunks of the routed groups' work, claimed from
// a grid-wide counter so that a CTA that is late or slow simply takes less.  The routed part
// needs the segment plan, which the preceding kernels write: next() calls
// griddepcontrol.wait once before it touches the plan (or before reporting the end).
//
// Routed work, range mode: positions (16 rows of one group for one of its segments, groups
// laid end to end); a chunk is a run of positions whose ends are moved to tile boundaries, its
// length shrinks as the work runs out (a third of the remaining per-CTA share, at least one
// tile).  Round-robin mode: a chunk is one (segment, tile, k chunk) item; consecutive items are
// the tiles of one segment, which then run on many CTAs at once and share the segment's token
// rows in L2.
// Rows per segment of a group of n rows cut into nseg segments: equal shares rounded up to the
// 16-row unit of the token boxes (never more than the segment limit, since nseg = ceil(n /
// limit)).  Equal shares instead of "full segments and a remainder": the instruction time
// follows the rows of a segment with a floor of about 64 rows, so 320 rows cost less as
// 160 + 160 than as 256 + 64.
__device__ __forceinline__ int balanced_segment_rows(int n, int nseg)
{
    return (((n + nseg - 1) / nseg) + 15) & ~15;
}

struct ItemWalk {
    const FfnArgs &a;
    const ClaimRing &ring;
    const bool claimer;    // this thread claims; all others follow the ring
    const bool lead;       // this thread arrives on the ring's barriers for its role
    const bool warp_wide;  // the role is run by all 32 lanes in lock step (epilogue warps)
    const int max_units;
    int n_claims;
    // shared expert: units (tile, k chunk, segment) sj, sj + grid, ...
    int sj, Us, s_base, s_rem, nseg_s, s_units;
    // routed groups: current chunk from (fs, u) to (fs_hi, u_hi); fs = plan index of a
    // group's first segment
    int R0, nseg_total, fs, u, fs_hi, u_hi;
    long long P;
    int ntiles;
    bool synced, group_loaded, have_chunk, finished, end_published;
    int n_pub;  // claimer: chunks published so far
    // current group and tile
    Segment sg;
    int g_nseg, g_u_end;
    bool have_tile;
    int t_grp, t_expert, t_u0, t_h, t_row0, t_n, t_s, t_s_end, t_seg0, t_seg_rows;
    bool t_once;  // the tile's weights are read by this pass over it only
    int t_k0, t_k1;
    long long t_out_off;

    __device__ ItemWalk(const FfnArgs &args, const ClaimRing &r, bool is_claimer, bool is_lead,
                        bool is_warp_wide, bool already_synced)
        : a(args), ring(r), claimer(is_claimer), lead(is_lead), warp_wide(is_warp_wide),
          max_units(args.max_tile >> 4),
          n_claims(0), synced(false), group_loaded(false), have_chunk(false), finished(false),
          end_published(false), n_pub(0),
          have_tile(false)
    {
        Us = a.with_shared ? a.rows[1] >> 4 : 0;
        s_base = a.shared_tiles ? Us / a.shared_tiles : 0;
        s_rem = a.shared_tiles ? Us % a.shared_tiles : 0;
        sj = blockIdx.x;
        nseg_s = (a.T + a.shared_seg - 1) / a.shared_seg;
        s_units = a.shared_tiles * a.shared_ksplit * nseg_s;
        R0 = a.rows[0] >> 4;
        nseg_total = fs = u = fs_hi = u_hi = 0;
        ntiles = (R0 + max_units - 1) / max_units;
        P = 0;
        if (already_synced)
            sync(false);
    }
    // position p -> (group, row unit rounded down to a tile boundary of the group)
    __device__ void boundary(long long p, int &fs_out, int &u_out) const
    {
        if (p >= P) {
            fs_out = nseg_total;
            u_out = 0;
            return;
        }
        const Segment s = a.seg[(int)(p / R0)];
        const int ns = (s.n + a.seg_rows - 1) / a.seg_rows;
        fs_out = s.first_seg;
        u_out = (int)((p - (long long)s.first_seg * R0) / ns) / max_units * max_units;
    }
    __device__ void sync(bool wait)
    {
        if (wait)
            griddep_wait();
        nseg_total = a.plan_header[0];
        P = a.round_robin ? (long long)a.plan_header[1] * ntiles * a.routed_ksplit
                          : (long long)nseg_total * R0;
        synced = true;
    }
    // Claims the next chunk from the grid-wide counter (claimer only).  In round-robin mode
    // the first item of every CTA is fixed -- item gridDim.x - 1 - blockIdx.x, so that the CTAs
    // without a shared-expert tile (the high ones) take the first routed items -- and costs no
    // round trip to the counter; the counter hands out the items from gridDim.x on.
    __device__ void claim(int &lo, int &hi)
    {
        if (a.round_robin) {
            lo = n_pub == 0 ? (int)(gridDim.x - 1 - blockIdx.x)
                            : (int)gridDim.x + atomicAdd(a.claim_counter, 1);
            hi = lo + 1;
        } else {
            const long long left = P - *reinterpret_cast<volatile int32_t *>(a.claim_counter);
            const long long guided = left / (3 * (long long)gridDim.x);
            const int size = (int)(guided > max_units ? guided : max_units);
            lo = atomicAdd(a.claim_counter, size);
            hi = (int)(lo + (long long)size < P ? lo + size : P);
        }
        if (lo >= P)
            lo = hi = -1;
    }
    // Claimer: claims one more chunk and publishes it in the ring (with its group looked up
    // in round-robin mode, so that the other roles need not go to global memory for it).
    __device__ bool publish_one()
    {
        const int slot = n_pub % FF_CLAIMS;
        const uint32_t par = (uint32_t)(n_pub / FF_CLAIMS) & 1u;
        int lo, hi, sidx = 0;
        Segment grp = sg;
        claim(lo, hi);
        if (lo >= 0 && a.round_robin) {
            // the pair entry carries its group: one load level between the claim and the tile
            const int4 *pe = reinterpret_cast<const int4 *>(a.pairs + lo / (ntiles * a.routed_ksplit));
            const int4 g = pe[0];
            sidx = pe[1].x;
            grp.expert = g.x;
            grp.row0 = g.y;
            grp.n = g.z;
            grp.first_seg = g.w;
        }
        if (!mbar_wait(ring.empty0 + 8u * slot, par ^ 1u, ring.abort_flag, ring.status))
            return false;
        int *e = ring.data + slot * FF_CLAIM_WORDS;
        e[0] = lo;
        e[1] = hi;
        e[2] = sidx;
        e[3] = grp.expert;
        e[4] = grp.row0;
        e[5] = grp.n;
        e[6] = grp.first_seg;
        __threadfence_block();
        mbar_arrive(ring.full0 + 8u * slot);
        ++n_pub;
        if (lo < 0)
            end_published = true;
        return true;
    }
    // Next chunk [lo, hi) of the routed work; false when none is left (or on abort).  In
    // round-robin mode the chunk is one item and `grp` receives its group.  While plenty of
    // work is left the claimer publishes one chunk beyond the one it is about to work on, so
    // that every role knows its next item before it finishes the current one (near the end a
    // chunk held in reserve would starve another CTA).
    __device__ bool acquire(int &lo, int &hi, Segment &grp, int &sidx)
    {
        const int slot = n_claims % FF_CLAIMS;
        const uint32_t par = (uint32_t)(n_claims / FF_CLAIMS) & 1u;
        int *e = ring.data + slot * FF_CLAIM_WORDS;
        if (claimer) {
            for (;;) {
                // (the counter is only read where the answer can be yes)
                const long long ample = 4 * (long long)gridDim.x * (a.round_robin ? 1 : max_units);
                const bool plenty =
                    P > ample && P - *reinterpret_cast<volatile int32_t *>(a.claim_counter) > ample;
                if (end_published || n_pub >= n_claims + (plenty ? 2 : 1))
                    break;
                if (!publish_one())
                    return false;
            }
        } else if (!mbar_wait(ring.full0 + 8u * slot, par, ring.abort_flag, ring.status)) {
            return false;
        }
        ++n_claims;
        lo = e[0];
        hi = e[1];
        sidx = e[2];
        grp.expert = e[3];
        grp.row0 = e[4];
        grp.n = e[5];
        grp.first_seg = e[6];
        if (!claimer) {
            if (warp_wide)
                __syncwarp();  // every lane has read the entry before it is released
            if (lead)
                mbar_arrive(ring.empty0 + 8u * slot);
        }
        return lo >= 0;
    }
    // false when this CTA has no further item
    __device__ bool next(Item &it)
    {
        for (;;) {
            if (have_tile) {
                if (t_s < t_s_end) {
                    it.grp = t_grp;
                    it.expert = t_expert;
                    it.f0 = t_u0 << 4;
                    it.h = t_h << 4;
                    it.row0 = t_row0 + t_s * t_seg_rows;
                    it.n = min(t_seg_rows, t_n - t_s * t_seg_rows);
                    it.seg = t_seg0 + t_s;
                    it.w_once = t_once;
                    it.k0 = t_k0;
                    it.k1 = t_k1;
                    it.out_off = t_out_off;
                    ++t_s;
                    return true;
                }
                have_tile = false;
            }
            if (sj < s_units) {  // next unit of the shared expert: (tile, k chunk, segment)
                const int tc = sj / nseg_s, q = sj - tc * nseg_s;
                const int tile = tc / a.shared_ksplit, chunk = tc - tile * a.shared_ksplit;
                t_k0 = chunk * a.shared_kchunk;
                t_k1 = min(a.K[1], t_k0 + a.shared_kchunk);
                t_out_off = chunk * a.shared_part_stride;
                t_u0 = tile * s_base + min(tile, s_rem);
                t_h = s_base + (tile < s_rem ? 1 : 0);
                t_grp = 1;
                t_expert = 0;
                t_row0 = 0;
                t_seg0 = 0;
                t_n = a.T;
                t_seg_rows = balanced_segment_rows(a.T, nseg_s);
                t_s = q;
                t_s_end = q + 1;
                t_once = nseg_s <= 1;
                sj += gridDim.x;
                have_tile = true;
                continue;
            }
            if (!synced)
                sync(true);
            if (finished)
                return false;
            if (!have_chunk) {
                int lo, hi, sidx;
                if (!acquire(lo, hi, sg, sidx)) {
                    finished = true;
                    return false;
                }
                if (a.round_robin) {
                    // one (segment, tile, k chunk) item
                    const int chunk = lo % a.routed_ksplit;
                    const int tile = (lo / a.routed_ksplit) % ntiles;
                    g_nseg = (sg.n + a.seg_rows - 1) / a.seg_rows;
                    t_u0 = tile * max_units;
                    t_h = min(max_units, R0 - t_u0);
                    t_grp = 0;
                    t_expert = sg.expert;
                    t_row0 = sg.row0;
                    t_seg0 = sg.first_seg;
                    t_n = sg.n;
                    t_seg_rows = balanced_segment_rows(sg.n, g_nseg);
                    t_s = sidx - sg.first_seg;
                    t_s_end = t_s + 1;
                    t_once = g_nseg <= 1;
                    t_k0 = chunk * a.routed_kchunk;
                    t_k1 = min(a.K[0], t_k0 + a.routed_kchunk);
                    t_out_off = chunk * a.routed_part_stride;
                    have_tile = true;
                    continue;
                }
                boundary(lo, fs, u);
                boundary(hi, fs_hi, u_hi);
                group_loaded = false;
                have_chunk = true;
            }
            if (fs >= nseg_total || fs > fs_hi || (fs == fs_hi && u >= u_hi)) {
                have_chunk = false;  // chunk exhausted (or empty after rounding)
                continue;
            }
            if (!group_loaded) {
                sg = a.seg[fs];
                g_nseg = (sg.n + a.seg_rows - 1) / a.seg_rows;
                g_u_end = fs == fs_hi ? u_hi : R0;
                group_loaded = true;
            }
            if (u < g_u_end) {  // next tile of this group, all its segments
                t_h = min(max_units, g_u_end - u);
                t_grp = 0;
                t_expert = sg.expert;
                t_u0 = u;
                t_row0 = sg.row0;
                t_seg0 = sg.first_seg;
                t_n = sg.n;
                t_seg_rows = balanced_segment_rows(sg.n, g_nseg);
                t_s = 0;
                t_s_end = g_nseg;
                t_once = g_nseg <= 1;
                t_k0 = 0;
                t_k1 = a.K[0];
                t_out_off = 0;
                u += t_h;
                have_tile = true;
                continue;
            }
            fs += g_nseg;  // group done: on to the next one
            u = 0;
            group_loaded = false;
        }
    }
};

// Placement of the token-ring entries.  An entry takes `m` consecutive units and never wraps:
// when it does not fit before the end of the ring it starts at unit 0.  Producer and MMA
// issuer replay the same sequence of sizes, so they agree on every position.
struct XRingWalk {
    int units, cur, count;
    __device__ XRingWalk(int n_units) : units(n_units), cur(0), count(0) {}
    // returns the first unit of the next entry; `pad` = units skipped at the end of the ring
    __device__ int place(int m, int &pad)
    {
        pad = 0;
        if (cur + m > units) {
            pad = units - cur;  // may be 0 when the previous entry ended exactly at the end
            cur = 0;
        }
        const int at = cur;
        cur += m;
        ++count;
        return at;
    }
};

__device__ __forceinline__ int pieces16(int n) { return (n + 15) >> 4; }

// One output value of an epilogue thread: h = silu(g) * u (GATED) or the plain sum, as bf16.
template <bool GATED>
__device__ __forceinline__ __nv_bfloat16 epilogue_value(uint32_t g, uint32_t u)
{
    float v = __uint_as_float(g);
    if (GATED)
        v = silu_f(v) * __uint_as_float(u);
    return __float2bfloat16_rn(v);
}

// Epilogue transposition.  An epilogue thread owns one output feature (its TMEM lane) and
// holds that feature's values for 16 consecutive tokens, but the outputs are token-major
// (features contiguous).  Two-byte stores of single values cost a fifth of the whole pass at
// large token counts, so the warp first exchanges values with three rounds of shuffles
// (lane distances 1, 2, 4): afterwards every lane holds, for two of the 16 tokens, eight
// consecutive features as one 16-byte vector.
//   in:  w[c]  bf16 bits (low half) of this lane's feature for token c, c = 0..15
//   out: v[i]  features 8*(lane>>3) .. +7 of token  tok[i],  i = 0, 1
__device__ __forceinline__ void transpose_16x32(const uint32_t (&w)[16], int lane, uint4 (&v)[2],
                                                int (&tok)[2])
{
    const bool b1 = lane & 1, b2 = lane & 2, b4 = lane & 4;
    // distance 1: pairs of features; even lanes keep tokens 0-7, odd lanes tokens 8-15
    uint32_t p[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t keep = b1 ? w[8 + i] : w[i];
        const uint32_t send = b1 ? w[i] : w[8 + i];
        const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 1);
        p[i] = b1 ? (recv | (keep << 16)) : (keep | (recv << 16));
    }
    // distance 2: four features; the lane of the lower pair keeps the first four of its tokens
    uint32_t q0[4], q1[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t keep = b2 ? p[4 + i] : p[i];
        const uint32_t send = b2 ? p[i] : p[4 + i];
        const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 2);
        q0[i] = b2 ? recv : keep;
        q1[i] = b2 ? keep : recv;
    }
    // distance 4: eight features, two tokens
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const uint32_t k0 = b4 ? q0[2 + i] : q0[i], k1 = b4 ? q1[2 + i] : q1[i];
        const uint32_t s0 = b4 ? q0[i] : q0[2 + i], s1 = b4 ? q1[i] : q1[2 + i];
        const uint32_t r0 = __shfl_xor_sync(0xffffffffu, s0, 4);
        const uint32_t r1 = __shfl_xor_sync(0xffffffffu, s1, 4);
        v[i] = b4 ? make_uint4(r0, r1, k0, k1) : make_uint4(k0, k1, r0, r1);
        tok[i] = (b1 ? 8 : 0) + (b2 ? 4 : 0) + (b4 ? 2 : 0) + i;
    }
}

// GATED: W_gate and W_up tiles -> h = silu(g) * u.   !GATED: W_down tiles -> y.
template <bool GATED>
__global__ void __launch_bounds__(FF_THREADS, 1)
ffn_fused_kernel(const FfnArgs args, const __grid_constant__ FfnMaps maps)
{
    constexpr int NW = GATED ? 2 : 1;  // weight matrices per tile (gate and up: one block each)

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * FF_MAX_W_SLOTS + 2 * FF_X_ENTRIES + 4 + 2 * FF_CLAIMS];
    __shared__ uint32_t tmem_base_holder;
    __shared__ int abort_flag[2];  // [0] raised by the first wait that gives up, [1] wait limit (us)
    __shared__ int claim_data[FF_CLAIMS * FF_CLAIM_WORDS];

    const int NS = args.n_w_slots;
    const int kb = args.kboxes;
    // TMEM: a set of accumulators is two blocks (gate and up, or two blocks of 128 down rows) of
    // acc_block columns each; two sets of 2 x 128 columns, or one set of 2 x 256
    const int acc_sets = args.acc_sets;
    const uint32_t acc_block = acc_sets == 2 ? 128u : 256u;
    // token ring first (an MMA reads exactly the rows of its entry, rounded up to 16; a weight
    // block is read as 128 rows, which for a shorter tile ends inside the slot's capacity)
    const uint32_t ring_x = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle needs 1 KB alignment
    const uint32_t ring_w = ring_x + (uint32_t)args.x_units * FF_X_UNIT;
    const uint32_t bar0 = smem_u32(bars);
    auto w_full = [&](int s) { return bar0 + 8u * s; };
    auto w_empty = [&](int s) { return bar0 + 8u * (FF_MAX_W_SLOTS + s); };
    auto x_full = [&](int s) { return bar0 + 8u * (2 * FF_MAX_W_SLOTS + s); };
    auto x_empty = [&](int s) { return bar0 + 8u * (2 * FF_MAX_W_SLOTS + FF_X_ENTRIES + s); };
    auto acc_full = [&](int b) { return bar0 + 8u * (2 * FF_MAX_W_SLOTS + 2 * FF_X_ENTRIES + b); };
    auto acc_empty = [&](int b) { return bar0 + 8u * (2 * FF_MAX_W_SLOTS + 2 * FF_X_ENTRIES + 2 + b); };
    const uint32_t claim_full0 = bar0 + 8u * (2 * FF_MAX_W_SLOTS + 2 * FF_X_ENTRIES + 4);
    const uint32_t claim_empty0 = claim_full0 + 8u * FF_CLAIMS;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag[0] = 0;
        abort_flag[1] = args.wait_us;
        for (int s = 0; s < NS; ++s) {
            mbar_init(w_full(s), 1);
            mbar_init(w_empty(s), 1);
        }
        for (int s = 0; s < FF_X_ENTRIES; ++s) {
            mbar_init(x_full(s), 1);
            mbar_init(x_empty(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full(b), 1);
            mbar_init(acc_empty(b), FF_EPI_WARPS);
        }
        for (int i = 0; i < FF_CLAIMS; ++i) {
            mbar_init(claim_full0 + 8u * i, 1);
            mbar_init(claim_empty0 + 8u * i, FF_CLAIM_READERS);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32(&tmem_base_holder)),
                     "r"(FF_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_holder;
    volatile int *abortp = abort_flag;
    const ClaimRing claims{claim_data, claim_full0, claim_empty0, abortp, args.status};

    if (warp == 0) {
        // ---------------- weight producer ----------------
        if (lane == 0) {
            // gate/up pass: the shared expert's weights and x are the caller's inputs, so those
            // items run before the wait.  Down pass: every weight tile may be fetched ahead --
            // the launch order guarantees that the plan is complete when this kernel starts.
            ItemWalk walk(args, claims, true, false, false, !GATED);
            const uint64_t pol_once = l2_policy_evict_first();
            bool launched = !GATED;
            if (!GATED)
                griddep_launch();
            int slot = 0;
            uint32_t phase = 0;
            bool ok = true;
            Item it;
            while (ok && walk.next(it)) {
                if (!launched && walk.synced) {
                    griddep_launch();  // after the wait: dependents may rely on the plan
                    launched = true;
                }
                const int K = it.k1;
                const uint32_t tile_bytes = (uint32_t)it.h * 128u;
                const int wrow = it.expert * args.rows[0] + it.f0;  // expert = 0 for the shared kind
                for (int k0 = it.k0; k0 < K; k0 += 64 * kb) {
                    const int nbox = min(kb, (K - k0 + 63) >> 6);
                    if (!mbar_wait(w_empty(slot), phase ^ 1u, abortp, args.status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t base = ring_w + slot * args.w_slot_bytes;
                    mbar_expect_tx(w_full(slot), nbox * NW * tile_bytes);
                    for (int b = 0; b < nbox; ++b) {
#pragma unroll
                        for (int m = 0; m < NW; ++m) {
                            // the tile as boxes of 128, 64, 32 and 16 rows, stacked
                            uint32_t dst = base + (uint32_t)(b * NW + m) * tile_bytes;
                            int row = wrow, rem = it.h;
                            while (rem > 0) {
                                const int hi = rem >= 128 ? 0 : (rem >= 64 ? 1 : (rem >= 32 ? 2 : 3));
                                const int bh = 128 >> hi;
                                if (it.w_once)
                                    tma_load_2d_hint(dst, &maps.w[it.grp][m][hi], w_full(slot), k0 + 64 * b,
                                                     row, pol_once);
                                else
                                    tma_load_2d(dst, &maps.w[it.grp][m][hi], w_full(slot), k0 + 64 * b, row);
                                dst += (uint32_t)bh * 128u;
                                row += bh;
                                rem -= bh;
                            }
                        }
                    }
                    if (++slot == NS) {
                        slot = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!walk.synced)
                walk.sync(true);
            if (!launched)
                griddep_launch();
        }
    } else if (warp == 2) {
        // ---------------- token-operand producer ----------------
        if (lane == 0) {
            // down pass: h is written by the preceding kernel, which may still be running; a
            // segment's rows are fetched once its progress counter says they are complete
            ItemWalk walk(args, claims, false, true, false, !GATED);
            XRingWalk ring(args.x_units);
            int seen = -1;  // (group kind, segment) key last found complete
            const uint64_t pol_keep = l2_policy_evict_last();
            int released = 0;          // entries known to have been consumed
            int v_cur = 0, v_rel = 0;  // virtual unit positions: issued up to / free up to
            int v_start_of[FF_X_ENTRIES];  // where each entry's rows begin (after its padding)
            bool ok = true;
            Item it;
            while (ok && walk.next(it)) {
                const int K = it.k1;
                if (!GATED) {
                    const int key = (it.grp << 30) | it.seg;
                    if (key != seen) {
                        // every epilogue warp of the gate/up pass counts the 16-column units
                        // of h it has finished for the segment
                        ok = counter_wait(args.done[it.grp] + it.seg, (args.K[it.grp] >> 4) * FF_EPI_WARPS, abortp,
                                          args.status);
                        seen = key;
                        if (!ok)
                            break;
                        // rows written through the generic proxy, read below by the async proxy
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                    }
                }
                const int pieces = pieces16(it.n);
                const int m = pieces * kb;
                for (int k0 = it.k0; ok && k0 < K; k0 += 64 * kb) {
                    const int nbox = min(kb, (K - k0 + 63) >> 6);
                    const int j = ring.count;
                    int pad;
                    const int at = ring.place(m, pad);
                    const int v_start = v_cur + pad, v_end = v_start + m;
                    // the entry's units (and its barrier pair) must have been released:
                    // everything before the oldest entry still in use is free, the
                    // padding in front of it included
                    while (released < j &&
                           (j - released >= FF_X_ENTRIES || v_end - v_rel > args.x_units)) {
                        const int r = released % FF_X_ENTRIES;
                        if (!mbar_wait(x_empty(r), (uint32_t)(released / FF_X_ENTRIES) & 1u, abortp,
                                       args.status)) {
                            ok = false;
                            break;
                        }
                        ++released;
                        v_rel = released < j ? v_start_of[released % FF_X_ENTRIES] : v_start;
                    }
                    if (!ok)
                        break;
                    const int e = j % FF_X_ENTRIES;
                    v_start_of[e] = v_start;
                    v_cur = v_end;
                    const uint32_t base = ring_x + (uint32_t)at * FF_X_UNIT;
                    mbar_expect_tx(x_full(e), (uint32_t)(nbox * pieces) * FF_X_UNIT);
                    for (int b = 0; b < nbox; ++b) {
                        // the entry's rows as boxes of 128, 64, 32 and 16 rows
                        uint32_t dst = base + (uint32_t)(b * pieces) * FF_X_UNIT;
                        int row = it.row0, rem = pieces << 4;
                        while (rem > 0) {
                            const int hi = rem >= 128 ? 0 : (rem >= 64 ? 1 : (rem >= 32 ? 2 : 3));
                            const int bh = 128 >> hi;
                            tma_load_2d_hint(dst, &maps.x[it.grp][hi], x_full(e), k0 + 64 * b, row,
                                             pol_keep);
                            dst += (uint32_t)bh * 128u;
                            row += bh;
                            rem -= bh;
                        }
                    }
                }
            }
            if (!walk.synced)
                walk.sync(true);
            if (!GATED)
                griddep_wait();  // no kernel of the chain completes before its predecessor
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            ItemWalk walk(args, claims, false, true, false, !GATED);
            XRingWalk ring(args.x_units);
            int sw = 0;
            uint32_t pw = 0;
            bool ok = true;
            int n_items = 0;
            Item it;
            while (ok && walk.next(it)) {
                // the accumulator set is waited for right before the item's first instruction, so
                // that its operands are already being fetched while the epilogue drains the set
                const int set = n_items % acc_sets;
                const uint32_t acc_par = ((uint32_t)(n_items / acc_sets) & 1u) ^ 1u;
                ++n_items;
                bool acc_ready = false;
                const uint32_t d0 = tmem_base + (uint32_t)set * 2u * acc_block;
                const uint32_t tile_bytes = (uint32_t)it.h * 128u;
                const int pieces = pieces16(it.n);
                const uint32_t idesc = umma_idesc_bf16(pieces << 4);  // M = 128, N = token rows
                // weight blocks of the tile: gate and up, or the 128-row halves of a down tile
                const int nblk = GATED ? 2 : (it.h + 127) >> 7;
                // descriptor steps in 16-byte units: to the next block, to the next k box
                const uint32_t blk16 = (GATED ? tile_bytes : 128u * 128u) >> 4;
                const uint64_t w_box16 = (uint64_t)((NW * tile_bytes) >> 4);
                const uint64_t x_box16 = (uint64_t)((pieces * FF_X_UNIT) >> 4);
                const int K = it.k1;
                for (int k0 = it.k0; ok && k0 < K; k0 += 64 * kb) {
                    const int nbox = min(kb, (K - k0 + 63) >> 6);
                    const int j = ring.count;
                    int pad;
                    const int at = ring.place(pieces * kb, pad);
                    const int xe = j % FF_X_ENTRIES;
                    const uint32_t xpar = (uint32_t)(j / FF_X_ENTRIES) & 1u;
                    const uint32_t xbase = ring_x + (uint32_t)at * FF_X_UNIT;
                    if (!mbar_wait(w_full(sw), pw, abortp, args.status) ||
                        !mbar_wait(x_full(xe), xpar, abortp, args.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    if (!acc_ready) {
                        if (!mbar_wait(acc_empty(set), acc_par, abortp, args.status)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        acc_ready = true;
                    }
                    uint64_t w_desc = umma_desc_sw128(ring_w + sw * args.w_slot_bytes);
                    uint64_t x_desc = umma_desc_sw128(xbase);
                    for (int b = 0; b < nbox; ++b) {
                        const uint32_t accum = ((k0 - it.k0) | b) != 0 ? 1u : 0u;
                        if (nblk == 2)
                            issue_k_box<2>(d0, acc_block, w_desc, blk16, x_desc, idesc, accum);
                        else
                            issue_k_box<1>(d0, acc_block, w_desc, blk16, x_desc, idesc, accum);
                        w_desc += w_box16;
                        x_desc += x_box16;
                    }
                    umma_commit(x_empty(xe));
                    umma_commit(w_empty(sw));  // reusable once these MMAs have read it
                    if (++sw == NS) {
                        sw = 0;
                        pw ^= 1u;
                    }
                }
                if (ok)
                    umma_commit(acc_full(set));  // accumulators complete
            }
            if (!walk.synced)
                walk.sync(true);
        }
    } else {
        // ---------------- epilogue (warps 3..10) ----------------
        // down pass: its outputs are read by nothing older than this call's combine, so the
        // stores need not wait for the preceding kernel (the token producer does, per segment)
        const int quarter = warp & 3;  // TMEM lanes 32*quarter .. +31 belong to this warp
        const int chunk0 = warp >= 7 ? 16 : 0;  // the quarter's second warp takes the odd chunks
        ItemWalk walk(args, claims, false, lane == 0, true, !GATED);
        int n_items = 0;
        Item it;
        for (;;) {
            // the walk is identical in all lanes; griddepcontrol.wait inside next() is
            // executed by every lane
            if (!walk.next(it))
                break;
            const int set = n_items % acc_sets;
            const uint32_t acc_phase = (uint32_t)(n_items / acc_sets) & 1u;
            ++n_items;
            // every lane waits; the vote makes the decision uniform and reconverges the warp
            // for the warp-collective tcgen05.ld below
            const bool ready = mbar_wait(acc_full(set), acc_phase, abortp, args.status);
            if (!__all_sync(0xffffffffu, ready))
                break;
            tc_fence_after();
            // a thread owns one weight row (output feature) of a block and walks the tokens
            const int nblk = GATED ? 1 : (it.h + 127) >> 7;  // gate and up are read together
            const int ld = args.out_ld[it.grp];
            const int npad = pieces16(it.n) << 4;
            for (int m = 0; m < nblk; ++m) {
                const int rows_blk = GATED ? it.h : min(128, it.h - 128 * m);
                if (quarter * 32 >= rows_blk)
                    break;  // this warp's lanes lie beyond the tile (uniform)
                // after the transposition this lane stores features 8 * (lane >> 3) .. + 7 of
                // the warp's 32 (tiles are multiples of 16 features: all eight exist or none)
                const int fgrp = quarter * 32 + 8 * (lane >> 3);
                const bool grp_ok = fgrp < rows_blk;
                __nv_bfloat16 *out = args.out[it.grp] + it.out_off + (size_t)it.row0 * ld + it.f0 +
                                     128 * m + fgrp;
                const uint32_t t0 = tmem_base + ((uint32_t)(quarter * 32) << 16) +
                                    (uint32_t)set * 2u * acc_block + (uint32_t)m * acc_block;
                // two register buffers: the TMEM load of this warp's next 16 tokens is in flight
                // while the current 16 are converted, transposed and stored
                uint32_t g[2][16], u[2][16];
                if (chunk0 < npad) {
                    tmem_ld16(t0 + chunk0, g[0]);
                    if (GATED)
                        tmem_ld16(t0 + acc_block + chunk0, u[0]);
                }
#pragma unroll 1
                for (int c = chunk0; c < npad; c += 64) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int cc = c + 32 * half;
                        if (cc < npad) {
                            tmem_ld_wait();
                            if (cc + 32 < npad) {
                                tmem_ld16(t0 + cc + 32, g[half ^ 1]);
                                if (GATED)
                                    tmem_ld16(t0 + acc_block + cc + 32, u[half ^ 1]);
                            }
                            uint32_t w[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const __nv_bfloat16 val = epilogue_value<GATED>(g[half][i], u[half][i]);
                                w[i] = (uint32_t)__bfloat16_as_ushort(val);
                            }
                            uint4 v[2];
                            int tok[2];
                            transpose_16x32(w, lane, v, tok);
#pragma unroll
                            for (int i = 0; i < 2; ++i)
                                if (grp_ok && cc + tok[i] < it.n)
                                    *reinterpret_cast<uint4 *>(out + (size_t)(cc + tok[i]) * ld) = v[i];
                        }
                    }
                }
            }
            tc_fence_before();
            if (GATED)  // the down pass fetches these rows with TMA (async proxy)
                asm volatile("fence.proxy.async.global;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(acc_empty(set));
                if (GATED) {
                    // publish: this warp's part of the tile is in h (a releasing reduction: the
                    // warp does not wait for its stores to become visible, the counter does)
                    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(args.done[it.grp] + it.seg),
                                 "r"(it.h >> 4)
                                 : "memory");
                }
            }
        }
        if (!walk.synced)
            walk.sync(true);
    }

    if (*abortp) {
        // A wait gave up.  Copies and tensor-core instructions already issued may still be in
        // flight: every thread that sees the flag (the one that raised it always does) holds
        // the CTA for a millisecond, far longer than any of them takes, before shared memory
        // and TMEM are given back.
        const uint64_t t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) {
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();  // lane 0 arrived from the issue loop: reconverge for the aligned dealloc
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"(FF_TMEM_COLS)
                     : "memory");
    }
}

// ---- self-test of the bounded wait ---------------------------------------------------------

// Waits, with the given limit, for a progress counter that nothing advances: the wait the down
// pass uses for the gate/up pass's counters must give up, raise the status word and return.
__global__ void wait_limit_selftest_kernel(int32_t *status, int32_t *never_set, int limit_us)
{
    __shared__ int abort_flag[2];
    if (threadIdx.x == 0) {
        abort_flag[0] = 0;
        abort_flag[1] = limit_us;
        status[0] = 0;
        status[1] = STATUS_MAGIC;
        never_set[0] = 0;
        __threadfence();
        counter_wait(never_set, 1, abort_flag, status);
    }
}

cudaError_t launch_wait_limit_selftest(int32_t *status, int32_t *never_set, int limit_us,
                                       cudaStream_t s)
{
    wait_limit_selftest_kernel<<<1, 32, 0, s>>>(status, never_set, limit_us);
    return cudaGetLastError();
}

// ---- gather of the token rows into sorted order (B operand of the gate/up pass) ---------

constexpr int GATHER_UNROLL = 8;

// One warp per sorted row: the source token is looked up once per row (all lanes read the same
// word), then the row is copied in passes of GATHER_UNROLL x 512 bytes whose loads are all in
// flight before the first store.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const __nv_bfloat16 *__restrict__ x, const int32_t *__restrict__ perm, int A,
                   int H, int top_k, __nv_bfloat16 *__restrict__ x_sorted)
{
    griddep_launch();
    griddep_wait();
    const int lane = threadIdx.x & 31;
    const int warps = (int)((gridDim.x * blockDim.x) >> 5);
    const int vec_per_row = H >> 3;
    for (int r = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5); r < A; r += warps) {
        const int t = perm[r] / top_k;
        const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)t * H);
        uint4 *dst = reinterpret_cast<uint4 *>(x_sorted + (size_t)r * H);
        for (int v0 = lane; v0 < vec_per_row; v0 += 32 * GATHER_UNROLL) {
            uint4 d[GATHER_UNROLL];
#pragma unroll
            for (int u = 0; u < GATHER_UNROLL; ++u)
                if (v0 + 32 * u < vec_per_row)
                    d[u] = src[v0 + 32 * u];
#pragma unroll
            for (int u = 0; u < GATHER_UNROLL; ++u)
                if (v0 + 32 * u < vec_per_row)
                    dst[v0 + 32 * u] = d[u];
        }
    }
}

cudaError_t launch_gather_rows(const moe_config_t &c, const __nv_bfloat16 *x, const int32_t *perm,
                               int T, __nv_bfloat16 *x_sorted, cudaStream_t s)
{
    const int A = T * c.top_k;
    const size_t total = (size_t)A * (c.hidden >> 3);
    // An FFN CTA does not start on an SM while a CTA of another kernel is resident there
    // (measured, whatever their shared-memory and register needs), so until this kernel has
    // finished the gate/up pass runs its shared-expert tiles only on the SMs this kernel
    // leaves alone.  Up to 16 MB of rows the gather therefore runs as one CTA per SM at most
    // (the hardware places them on about half of the SMs; fewer, larger CTAs made the gather
    // itself too slow); a large gather needs every SM's full thread count.
    size_t blocks = ((size_t)A + 7) / 8;  // a row per warp, eight warps per CTA
    const size_t cap = (size_t)sm_count() * (total * 16 <= (16u << 20) ? 1 : 8);
    if (blocks > cap)
        blocks = cap;
    return launch_pdl(gather_rows_kernel, dim3((unsigned)blocks), dim3(256), 0, s, x, perm, A,
                      c.hidden, c.top_k, x_sorted);
}

// ---- host side: geometry, tensor maps and launches ---------------------------------------

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

// 2-D bf16 tensor [rows, cols] (cols contiguous), box = 64 columns x box_rows, 128-byte swizzle.
bool make_tma_map_2d_bf16(CUtensorMap *m, const void *base, uint64_t rows, uint64_t cols,
                          uint32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn)
        return false;
    if (base == nullptr || rows == 0 || cols == 0) {
        memset(m, 0, sizeof *m);  // group kind not present: never used by the kernel
        return true;
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// the four box heights of one matrix
static bool make_weight_maps(CUtensorMap (&m)[FF_HEIGHTS], const void *base, uint64_t rows, uint64_t cols)
{
    for (int i = 0; i < FF_HEIGHTS; ++i)
        if (!make_tma_map_2d_bf16(&m[i], base, rows, cols, 128u >> i))
            return false;
    return true;
}

// Encoded tensor maps of recent launches.  A serving loop calls the layer with the same
// weights, workspace and token count again and again; encoding the twenty maps of a pass costs
// more host time than the launch itself, so the maps are kept, keyed by everything that enters
// them (device, pass, base pointers, extents).  A few dozen entries, replaced in turn.
struct MapKey {
    int device, gated;
    const void *ptr[7];
    uint64_t dim[6];
};
struct MapCacheEntry {
    bool used;
    MapKey key;
    FfnMaps maps;
};
constexpr int FF_MAP_CACHE = 48;
static MapCacheEntry g_map_cache[FF_MAP_CACHE];
static int g_map_cache_next = 0, g_map_cache_last = 0;
static std::mutex g_map_cache_mutex;

static bool map_cache_lookup(const MapKey &key, FfnMaps &out)
{
    std::lock_guard<std::mutex> lock(g_map_cache_mutex);
    for (int n = 0; n < FF_MAP_CACHE; ++n) {
        const int i = (g_map_cache_last + n) % FF_MAP_CACHE;  // the last hit first
        if (g_map_cache[i].used && memcmp(&g_map_cache[i].key, &key, sizeof key) == 0) {
            out = g_map_cache[i].maps;
            g_map_cache_last = i;
            return true;
        }
    }
    return false;
}

static void map_cache_store(const MapKey &key, const FfnMaps &maps)
{
    std::lock_guard<std::mutex> lock(g_map_cache_mutex);
    MapCacheEntry &e = g_map_cache[g_map_cache_next];
    e.used = true;
    e.key = key;
    e.maps = maps;
    g_map_cache_last = g_map_cache_next;
    g_map_cache_next = (g_map_cache_next + 1) % FF_MAP_CACHE;
}

static MapKey map_key(bool gated, const void *p0, const void *p1, const void *p2, const void *p3,
                      const void *p4, const void *p5, const void *p6, uint64_t d0, uint64_t d1,
                      uint64_t d2, uint64_t d3, uint64_t d4, uint64_t d5)
{
    MapKey k;
    memset(&k, 0, sizeof k);  // padding bytes take part in the comparison
    cudaGetDevice(&k.device);
    k.gated = gated ? 1 : 0;
    const void *p[7] = {p0, p1, p2, p3, p4, p5, p6};
    const uint64_t d[6] = {d0, d1, d2, d3, d4, d5};
    memcpy(k.ptr, p, sizeof p);
    memcpy(k.dim, d, sizeof d);
    return k;
}

// Expected number of activated experts for T tokens (Eq. N(t): E(1 - (1 - K/E)^T)); the host
// never sees the routing result, so it sizes rings and shared tiles from the expectation.
static double expected_active_experts(int E, int k, int T)
{
    return E * (1.0 - pow(1.0 - (double)k / E, (double)T));
}

static int ffn_grid() { return sm_count(); }

// Segment size of a call (the N limit of its tensor-core instructions).  Groups in the hundreds
// of rows want the contraction geometry: segments of 256 rows, so that a weight tile is fetched
// once per 256 tokens and the instruction runs at its full rate.  Small groups want the
// streaming geometry (segments of 128 rows, 64 KB weight slots, double-buffered accumulators).
// The host never sees the routing result, so it decides on the expected rows per group -- and on
// the shared expert, whose group is all T tokens: where its weights are a large part of the
// layer's, every extra segment is another pass over them through L2.
int ffn_segment_rows(const moe_config_t &c, int T)
{
    const int force = geometry_override();
    if (force >= 0)
        return force == 1 ? FF_SEG_WIDE : FF_SEG;
    if (T <= FF_SEG)
        return FF_SEG;
    // measured cross-over: about 112 expected rows per group (most groups then exceed one
    // 128-row segment), or a shared expert several times an expert's size
    const double rows_per_group = (double)T * c.top_k / expected_active_experts(c.n_experts, c.top_k, T);
    if (rows_per_group > 0.875 * FF_SEG)
        return FF_SEG_WIDE;
    return c.shared_inter >= 6 * c.inter ? FF_SEG_WIDE : FF_SEG;
}

// Up to 128 tokens no group of the layer has more than one 128-row segment and the token ring
// can be 32 KB, which leaves room for a third weight slot (worth 3-4 % of the layer) --
// provided the entries stay within half of the ring, i.e. 64 rows: always so up to 64 tokens;
// between 65 and 128 tokens only while the routed groups are expected to be small (a larger
// group still works, its rows are then not fetched ahead), and the shared expert's rows are
// then cut into two 64-row segments.
static bool small_token_ring(const moe_config_t &c, int T)
{
    if (T <= FF_SEG / 2)
        return true;
    if (T > FF_SEG)
        return false;
    // (a mean of up to a quarter of a segment: the largest group then stays within a half)
    return (double)T * c.top_k / expected_active_experts(c.n_experts, c.top_k, T) <= FF_SEG / 4 + 0.5;
}

// Token rows per segment of the shared expert (see small_token_ring).
static int shared_segment_rows(const moe_config_t &c, int T)
{
    if (T > FF_SEG / 2 && small_token_ring(c, T))
        return FF_SEG / 2;
    return ffn_segment_rows(c, T);
}

// Number of tiles the shared expert's rows are cut into.  The shared expert's work units are
// (tile, k chunk, segment); a unit should cost about the expected per-CTA share of the whole
// pass (or less), with the tile height within [min_tile, max_tile] rows (a weight block
// costs the same instruction time whether it holds 16 rows or 128).
static int shared_tile_count(const moe_config_t &c, int T, int rows_routed, int rows_shared,
                             int K_routed, int K_shared, int ksplit, int min_tile, int max_tile,
                             int grid)
{
    const int seg_s = shared_segment_rows(c, T), seg_r = ffn_segment_rows(c, T);
    const int nseg_s = (T + seg_s - 1) / seg_s;
    const int units = rows_shared >> 4;
    const double k_ratio = (double)K_shared / K_routed;  // cost of a shared row unit per segment
    const double n_act = expected_active_experts(c.n_experts, c.top_k, T);
    const double segs_r = n_act * ceil((double)T * c.top_k / n_act / seg_r);
    const double total = units * k_ratio * nseg_s + segs_r * (rows_routed >> 4);
    int tu = (int)ceil(total / grid / (k_ratio / ksplit));
    if (tu < (min_tile >> 4))
        tu = min_tile >> 4;
    if (tu > (max_tile >> 4))
        tu = max_tile >> 4;
    return (units + tu - 1) / tu;
}

// Ring geometry.  Streaming: two k boxes per weight slot (64 KB for a full tile: every row is
// fetched in 256 contiguous bytes, which both HBM and L2 serve markedly faster than 128); the
// token ring holds two entries of the largest possible segment while no group can exceed 64
// rows (32 KB, three weight slots), three 128-row entries otherwise (96 KB, two slots).
// Contraction: one k box per slot and per entry, three 256-row entries (96 KB), four slots.
static void ffn_geometry(const moe_config_t &c, int T, FfnArgs &a)
{
    a.seg_rows = ffn_segment_rows(c, T);
    const bool wide = a.seg_rows > FF_SEG;
    a.kboxes = wide ? 1 : 2;
    a.acc_sets = wide ? 1 : 2;
    a.w_slot_bytes = 256 * 128 * a.kboxes;  // a full tile: 256 rows per k box
    const int x_ring_bytes = (!wide && small_token_ring(c, T)) ? 32 * 1024 : 96 * 1024;
    a.x_units = x_ring_bytes / FF_X_UNIT;
    const int avail = FF_SMEM_LIMIT - 1024 - 512;  // alignment slack, static shared memory
    int ns = (avail - x_ring_bytes) / a.w_slot_bytes;
    if (ns > FF_MAX_W_SLOTS)
        ns = FF_MAX_W_SLOTS;
    a.n_w_slots = ns;
    a.wait_us = (int)(FF_WAIT_NS / 1000ull);
    a.shared_seg = shared_segment_rows(c, T);
}

// Range mode keeps every CTA alone on "its" groups, perfectly levelled.  It loses when
//  - a range is shorter than a few tiles: its two ends are partial tiles, and a weight block
//    costs K/16 tensor-core instructions whatever its height, so short ranges turn issue-bound;
//  - the token rows of `grid` groups do not fit in L2 beside the weight stream (large T): every
//    tile would fetch its group's rows from HBM again.
// Then, and when there are so many tiles per CTA that the last wave hardly matters, the routed
// work is dealt round-robin as (segment, tile) items: full tiles only, and the CTAs work on a
// few groups at a time.
static bool use_round_robin(const moe_config_t &c, int T, int rows_routed, int K_routed, int max_tile,
                            int grid)
{
    const int force = schedule_override();
    if (force >= 0)
        return force == 1;
    const double n_act = expected_active_experts(c.n_experts, c.top_k, T);
    const double rows_per_group = (double)T * c.top_k / n_act;
    const double segs = n_act * ceil(rows_per_group / ffn_segment_rows(c, T));
    const double tiles_per_cta = segs * ((rows_routed + max_tile - 1) / max_tile) / grid;
    const double token_bytes = rows_per_group * K_routed * 2.0 * grid;
    return tiles_per_cta < 3.0 || tiles_per_cta >= 12.0 || token_bytes > 200.0 * 1024 * 1024;
}

template <bool GATED>
static cudaError_t launch_ffn(FfnArgs &a, const FfnMaps &maps, cudaStream_t s)
{
    // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
    static DeviceOnce configured;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess)
        return cudaErrorInvalidDevice;
    if (!configured.done(dev)) {
        cudaError_t e = cudaFuncSetAttribute(ffn_fused_kernel<GATED>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             FF_SMEM_LIMIT - 512);
        if (e != cudaSuccess)
            return e;
        configured.mark(dev);
    }
    const size_t smem = (size_t)a.x_units * FF_X_UNIT + (size_t)a.n_w_slots * a.w_slot_bytes + 1024;
    if (a.n_w_slots < 2 || smem > FF_SMEM_LIMIT - 512)
        return cudaErrorInvalidConfiguration;
    return launch_pdl(ffn_fused_kernel<GATED>, dim3(ffn_grid()), dim3(FF_THREADS), smem, s, a, maps);
}

cudaError_t launch_ffn_gateup(const moe_config_t &c, const moe_weights_t &w, const __nv_bfloat16 *x,
                              const __nv_bfloat16 *x_sorted, int T, PlanView plan, bool with_shared,
                              __nv_bfloat16 *h, __nv_bfloat16 *h_shared, int32_t *status,
                              cudaStream_t s)
{
    const uint64_t A = (uint64_t)T * c.top_k, H = c.hidden, E = c.n_experts;
    FfnArgs a{};
    a.rows[0] = c.inter;
    a.rows[1] = c.shared_inter;
    a.K[0] = a.K[1] = c.hidden;
    a.max_tile = 128;
    a.shared_ksplit = 1;
    a.shared_kchunk = (c.hidden + 127) / 128 * 128;
    a.shared_tiles = with_shared ? shared_tile_count(c, T, c.inter, c.shared_inter, c.hidden, c.hidden,
                                                     1, 64, 128, ffn_grid())
                                 : 0;
    ffn_geometry(c, T, a);
    FfnMaps maps;
    const MapKey key = map_key(true, w.w_gate, w.w_up, x_sorted, with_shared ? w.ws_gate : nullptr,
                               with_shared ? w.ws_up : nullptr, with_shared ? x : nullptr, nullptr, E,
                               (uint64_t)c.inter, H, A, with_shared ? (uint64_t)c.shared_inter : 0,
                               (uint64_t)T);
    if (!map_cache_lookup(key, maps)) {
        memset(&maps, 0, sizeof maps);
        bool ok = make_weight_maps(maps.w[0][0], w.w_gate, E * c.inter, H) &&
                  make_weight_maps(maps.w[0][1], w.w_up, E * c.inter, H) &&
                  make_weight_maps(maps.x[0], x_sorted, A, H);
        if (with_shared)
            ok = ok && make_weight_maps(maps.w[1][0], w.ws_gate, c.shared_inter, H) &&
                 make_weight_maps(maps.w[1][1], w.ws_up, c.shared_inter, H) &&
                 make_weight_maps(maps.x[1], x, T, H);
        if (!ok)
            return cudaErrorInvalidValue;
        map_cache_store(key, maps);
    }
    a.out[0] = h;
    a.out[1] = h_shared;
    a.out_ld[0] = c.inter;
    a.out_ld[1] = c.shared_inter;
    a.plan_header = plan.header;
    a.seg = plan.seg;
    a.pairs = plan.pairs;
    a.claim_counter = plan.header + 2;
    a.done[0] = plan.done_routed;
    a.done[1] = plan.done_shared;
    a.round_robin = use_round_robin(c, T, c.inter, c.hidden, a.max_tile, ffn_grid()) ? 1 : 0;
    a.routed_ksplit = 1;
    a.routed_kchunk = c.hidden;
    a.status = status;
    a.T = T;
    a.with_shared = with_shared ? 1 : 0;
    return launch_ffn<true>(a, maps, s);
}

// Length of a k chunk when K is cut into about `parts` pieces (a multiple of the 128-column
// weight slot), and the number of non-empty chunks that length gives.
static int split_chunk(int K, int parts) { return ((K + parts - 1) / parts + 127) / 128 * 128; }
static int split_parts(int K, int parts) { return (K + split_chunk(K, parts) - 1) / split_chunk(K, parts); }

// Expected number of (segment, tile) items of the routed down pass (counted with the wide
// segments, so that it never decreases with T).
static double routed_down_items(const moe_config_t &c, int T)
{
    const double n_act = expected_active_experts(c.n_experts, c.top_k, T);
    const double rows_per_group = (double)T * c.top_k / n_act;
    return ceil(n_act) * ceil(rows_per_group / FF_SEG_WIDE) * ((c.hidden + 255) / 256);
}

// k chunks of the routed groups' down projection.  While the pass has fewer than about three
// (segment, tile) items per CTA -- few tokens, or few experts with long reductions -- some SMs
// have no weight stream to pull and one SM cannot pull a tile faster than a fraction of what
// HBM delivers, so the reduction is cut; each chunk writes its own plane of y and the combine
// adds the planes.  (Fewer than three items per CTA also means the pass deals single items.)
int routed_down_parts(const moe_config_t &c, int T)
{
    if (!use_round_robin(c, T, c.hidden, c.inter, 256, ffn_grid()))
        return 1;
    int parts = (int)ceil(3.0 * ffn_grid() / routed_down_items(c, T));
    const int cap = c.inter / 1024;  // chunks below half a megabyte cost more than they level
    if (parts > cap)
        parts = cap;
    if (parts > ROUTED_SPLIT_MAX_PARTS)
        parts = ROUTED_SPLIT_MAX_PARTS;
    return parts < 1 ? 1 : split_parts(c.inter, parts);
}

size_t routed_split_max_rows(const moe_config_t &c, int T)
{
    if (c.inter / 1024 < 2)
        return 0;
    // largest T' <= T whose item count still asks for more than one part
    auto split = [&](int t) { return routed_down_items(c, t) < 3.0 * ffn_grid(); };
    if (!split(1))
        return 0;
    int lo = 1, hi = T;  // split(lo) holds
    if (split(hi))
        return (size_t)hi * c.top_k;
    while (hi - lo > 1) {
        const int mid = lo + (hi - lo) / 2;
        if (split(mid))
            lo = mid;
        else
            hi = mid;
    }
    return (size_t)lo * c.top_k;
}

int shared_down_parts(const moe_config_t &c)
{
    // a chunk about as long as a routed expert's reduction, and no longer than 2560 columns
    int s = c.shared_inter / c.inter;
    if (s < c.shared_inter / 2560)
        s = c.shared_inter / 2560;
    if (s < 2)
        return 1;
    return split_parts(c.shared_inter, s > 8 ? 8 : s);
}

cudaError_t launch_ffn_down(const moe_config_t &c, const moe_weights_t &w, int T, PlanView plan,
                            bool with_shared, const __nv_bfloat16 *h, const __nv_bfloat16 *h_shared,
                            __nv_bfloat16 *y, __nv_bfloat16 *y_shared, int shared_parts,
                            int routed_parts, int32_t *status, cudaStream_t s)
{
    const uint64_t A = (uint64_t)T * c.top_k, H = c.hidden, E = c.n_experts;
    FfnArgs a{};
    a.rows[0] = a.rows[1] = c.hidden;
    a.K[0] = c.inter;
    a.K[1] = c.shared_inter;
    a.max_tile = 256;
    a.shared_ksplit = with_shared ? shared_parts : 1;
    a.shared_kchunk = with_shared ? split_chunk(c.shared_inter, a.shared_ksplit) : 128;
    a.shared_part_stride = (long long)T * c.hidden;
    a.shared_tiles = with_shared ? shared_tile_count(c, T, c.hidden, c.hidden, c.inter, c.shared_inter,
                                                     a.shared_ksplit, 128, 256, ffn_grid())
                                 : 0;
    ffn_geometry(c, T, a);
    FfnMaps maps;
    const MapKey key = map_key(false, w.w_down, h, with_shared ? w.ws_down : nullptr,
                               with_shared ? h_shared : nullptr, nullptr, nullptr, nullptr, E,
                               (uint64_t)c.inter, H, A, with_shared ? (uint64_t)c.shared_inter : 0,
                               (uint64_t)T);
    if (!map_cache_lookup(key, maps)) {
        memset(&maps, 0, sizeof maps);
        bool ok = make_weight_maps(maps.w[0][0], w.w_down, E * H, c.inter) &&
                  make_weight_maps(maps.x[0], h, A, c.inter);
        if (with_shared)
            ok = ok && make_weight_maps(maps.w[1][0], w.ws_down, H, c.shared_inter) &&
                 make_weight_maps(maps.x[1], h_shared, T, c.shared_inter);
        if (!ok)
            return cudaErrorInvalidValue;
        map_cache_store(key, maps);
    }
    a.out[0] = y;
    a.out[1] = y_shared;
    a.out_ld[0] = a.out_ld[1] = c.hidden;
    a.plan_header = plan.header;
    a.seg = plan.seg;
    a.pairs = plan.pairs;
    a.claim_counter = plan.header + 3;
    a.done[0] = plan.done_routed;
    a.done[1] = plan.done_shared;
    a.round_robin = use_round_robin(c, T, c.hidden, c.inter, a.max_tile, ffn_grid()) ? 1 : 0;
    if (routed_parts > 1 && !a.round_robin)
        return cudaErrorInvalidValue;  // planes exist only where single items are dealt
    a.routed_ksplit = routed_parts;
    a.routed_kchunk = split_chunk(c.inter, routed_parts);
    if ((long long)(routed_parts - 1) * a.routed_kchunk >= c.inter ||
        (with_shared && (long long)(a.shared_ksplit - 1) * a.shared_kchunk >= c.shared_inter))
        return cudaErrorInvalidValue;  // an empty chunk would leave its plane unwritten
    a.routed_part_stride = (long long)A * c.hidden;
    a.status = status;
    a.T = T;
    a.with_shared = with_shared ? 1 : 0;
    return launch_ffn<false>(a, maps, s);
}

}  // namespace moe

"""Model of how the FFN kernels hand out the routed work (CPU only).

`ffn_fused_kernel` lays the weight rows of all routed groups end to end -- one position =
16 weight rows of one group for one of its segments (128 or 256 token rows, fixed per call) --
and its CTAs claim chunks [lo, hi) of positions from a grid-wide counter.  A chunk's two ends
are mapped to (group, row unit) and moved down to a tile boundary of that group; inside its
chunk a CTA processes whole tiles, each for all segments of the group.  This test replays that
rule for random groups and random claim sizes and checks what the kernels rely on: every
(group, tile) is processed by exactly one chunk, whatever the claim sizes, and in round-robin
mode every (segment, tile, k chunk) item exactly once.

It restates `ItemWalk::boundary`, the range walk of `ItemWalk::next` and `ItemWalk::claim`
(csrc/ffn_fused.cu) in Python: a change to those functions has to be made here as well.
"""
import random

SEG = 128   # set per test: the segment size of the call


def n_segments(rows):
    return (rows + SEG - 1) // SEG


def boundary(p, groups, first_seg, R0, max_units, P, nseg_total):
    """Position -> (plan index of the group's first segment, row unit rounded down to a tile)."""
    if p >= P:
        return nseg_total, 0
    seg = p // R0                     # plan segment the position falls into
    g = max(i for i, fs in enumerate(first_seg) if fs <= seg)
    ns = n_segments(groups[g])
    u = ((p - first_seg[g] * R0) // ns) // max_units * max_units
    return first_seg[g], u


def tiles_of_chunk(lo, hi, groups, first_seg, R0, max_units):
    nseg_total = sum(n_segments(r) for r in groups)
    P = nseg_total * R0
    fs, u = boundary(lo, groups, first_seg, R0, max_units, P, nseg_total)
    fs_hi, u_hi = boundary(hi, groups, first_seg, R0, max_units, P, nseg_total)
    out = []
    while not (fs >= nseg_total or fs > fs_hi or (fs == fs_hi and u >= u_hi)):
        g = first_seg.index(fs)
        u_end = u_hi if fs == fs_hi else R0
        while u < u_end:
            h = min(max_units, u_end - u)
            out.append((g, u, h))
            u += h
        fs += n_segments(groups[g])
        u = 0
    return out


def test_every_tile_is_claimed_exactly_once_in_range_mode():
    global SEG
    rng = random.Random(7)
    for trial in range(300):
        SEG = 128 if trial % 2 else 256
        R0 = rng.choice([88, 160, 128, 37])            # 16-row units of weight rows per group
        max_units = rng.choice([8, 16])
        groups = [rng.choice([1, 5, 16, 100, 128, 129, 200, 257, 400]) for _ in range(rng.randint(1, 12))]
        first_seg, acc = [], 0
        for r in groups:
            first_seg.append(acc)
            acc += n_segments(r)
        P = acc * R0
        seen = {}
        lo = 0
        while lo < P:
            size = rng.choice([max_units, max_units, 3 * max_units, rng.randint(1, 4 * R0)])
            hi = min(P, lo + size)
            for g, u, h in tiles_of_chunk(lo, hi, groups, first_seg, R0, max_units):
                assert h > 0 and u % max_units == 0
                for unit in range(u, u + h):
                    assert (g, unit) not in seen, "row unit claimed twice"
                    seen[(g, unit)] = 1
            lo = hi
        assert len(seen) == len(groups) * R0, "row units missing"


def test_round_robin_items_cover_every_segment_tile_and_k_chunk_once():
    rng = random.Random(8)
    for _ in range(200):
        grid = rng.choice([4, 148])
        ntiles = rng.randint(1, 23)
        ksplit = rng.randint(1, 8)
        nsegs = rng.randint(1, 40)
        P = nsegs * ntiles * ksplit
        items = []
        counter = 0
        ctas = list(range(grid))
        rng.shuffle(ctas)
        active = set(ctas)
        first = {b: True for b in ctas}
        while active:
            b = rng.choice(sorted(active))
            if first[b]:                      # every CTA's first item is fixed
                lo = grid - 1 - b
                first[b] = False
            else:                             # the counter hands out the items from `grid` on
                lo = grid + counter
                counter += 1
            if lo >= P:
                active.discard(b)
                continue
            items.append((lo // (ntiles * ksplit), (lo // ksplit) % ntiles, lo % ksplit))
        assert len(items) == P and len(set(items)) == P

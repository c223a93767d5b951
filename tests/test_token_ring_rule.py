"""Model of the FFN kernels' token ring (CPU only).

The token-operand ring of `ffn_fused_kernel` holds entries of 2 KB units that never wrap: an
entry that does not fit before the end of the ring starts at unit 0, and the producer may place
entry j once everything before the oldest entry still in use is free.  The MMA side consumes
one entry per k step.  This test replays that rule over random item sequences: the geometries
the host chooses -- 48 units for segments of up to 16 units (128 rows at two k boxes per entry,
or 256 rows at one), 16 units for batches of up to 128 tokens -- never stall and never overlap
live entries.

It restates `XRingWalk::place` and the release loop of the token producer (csrc/ffn_fused.cu)
in Python: a change to those has to be made here as well.
"""
import random

ENTRIES = 8  # barrier pairs = entries in flight


def replay(units, steps):
    """steps: list of lists of entry sizes consumed together.  Returns 'ok', 'stall' or
    'overlap'."""
    seq = [m for st in steps for m in st]
    first_of_step = []
    acc = 0
    for st in steps:
        first_of_step.append(acc)
        acc += len(st)
    cur = 0          # next free physical unit
    v_cur = 0        # virtual position issued up to (physical position + laps * units)
    v_rel = 0        # virtual position free up to
    released = 0     # entries the producer knows to be consumed
    v_start = {}     # virtual start of every issued entry's rows
    live = {}        # entry -> (physical start, size), until released
    issued = consumed_entries = consumed_steps = 0
    while consumed_steps < len(steps):
        progressed = False
        if issued < len(seq):
            j, m = issued, seq[issued]
            pad, at = 0, cur
            if at + m > units:
                pad, at = units - cur, 0
            start, end = v_cur + pad, v_cur + pad + m
            rel, vr = released, v_rel
            blocked = False
            while rel < j and (j - rel >= ENTRIES or end - vr > units):
                if rel < consumed_entries:   # its MMAs have completed
                    rel += 1
                    vr = v_start[rel] if rel < j else start
                else:
                    blocked = True
                    break
            released, v_rel = rel, vr
            for q in [q for q in live if q < released]:
                del live[q]
            if not blocked:
                for a2, m2 in live.values():
                    if not (at + m <= a2 or a2 + m2 <= at):
                        return "overlap"
                live[j] = (at, m)
                v_start[j] = start
                v_cur, cur = end, at + m
                issued += 1
                progressed = True
        s = consumed_steps
        if first_of_step[s] + len(steps[s]) <= issued:
            consumed_entries += len(steps[s])
            consumed_steps += 1
            progressed = True
        if not progressed:
            return "stall"
    return "ok"


def random_steps(rng, max_units, even):
    """Items as the kernels produce them: one entry per k step, all k steps of an item of the
    same size (even in the streaming geometry: two k boxes per entry)."""
    steps = []
    for _ in range(rng.randint(1, 8)):
        k_steps = rng.randint(1, 6)
        m = rng.randint(1, max_units // 2) * 2 if even else rng.randint(1, max_units)
        steps += [[m]] * k_steps
    return steps


def test_large_ring_never_stalls():
    """96 KB: entries of up to 16 units (a full segment in either geometry)."""
    rng = random.Random(1)
    for _ in range(4000):
        assert replay(48, random_steps(rng, 16, True)) == "ok"
    for _ in range(4000):
        assert replay(48, random_steps(rng, 16, False)) == "ok"


def test_small_ring_never_stalls():
    """Up to 128 tokens: entries of up to half the ring (the shared expert's 64-row segments,
    groups of up to 64 rows) or, for a routed group of up to 128 rows, of the whole ring."""
    rng = random.Random(2)
    for _ in range(4000):
        assert replay(16, random_steps(rng, 8, True)) == "ok"
    for _ in range(4000):
        assert replay(16, random_steps(rng, 16, True)) == "ok"


def test_entries_in_flight_are_bounded_by_the_barrier_pairs():
    # many tiny entries: the eight barrier pairs, not the space, limit the producer
    assert replay(48, [[2]] * 100) == "ok"

"""Randomised parity: moe_verify_layer against the oracle on seeded random shapes.

Every case draws a layer shape (hidden, experts, top-k, intermediate sizes, score function,
renormalisation, shared expert and its gate, routing skew) and a token count around the
boundaries the kernels care about (1, 32/33 tokens, 64/65, 128/129 rows, several segments),
then runs the full comparison: logits, bit-exact routing and grouping, outputs within the
stated tolerance.
"""
import random

import pytest

from paper_2505_19645_b200 import workloads as wl
from parity_utils import check_layer_against_oracle

pytestmark = pytest.mark.gpu

CASES_PER_SEED = 200


def draw_case(rng):
    while True:
        H = 32 * rng.choice([1, 2, 3, 4, 5, 8, 9, 16, 17, 24, 32])
        E = rng.choice([1, 2, 3, 5, 8, 16, 24, 60, 64, 100, 256, 512])
        k = min(E, rng.choice([1, 1, 2, 2, 3, 4, 6, 8, 12, 16]))
        I = 32 * rng.choice([1, 2, 3, 4, 7, 8, 11, 16, 33, 64, 80])
        Is = 32 * rng.choice([0, 0, 1, 3, 4, 8, 13, 44, 96])
        score = rng.choice([0, 1])
        renorm = rng.choice([0, 1])
        sgate = rng.choice([0, 1]) if Is else 0
        zipf = rng.choice([None, None, 1.0, 1.2])
        t_max = 700 if k <= 4 else 300
        T = rng.choice([1, 2, 3, 5, 8, 16, 31, 32, 33, 64, 65, 96, 127, 128, 129, 130, 200, 256,
                        257, rng.randint(1, t_max), rng.randint(1, t_max)])
        # keep the oracle within a fraction of a second and the weights within a gigabyte
        if T * k * max(I, H) > 20_000_000 or T * max(Is, 1) * H > 100_000_000:
            continue
        if E * I * H * 6 > 1_000_000_000:
            continue
        return H, E, k, I, Is, score, renorm, sgate, zipf, T


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_match_the_oracle(seed):
    rng = random.Random(seed)
    for n in range(CASES_PER_SEED):
        H, E, k, I, Is, score, renorm, sgate, zipf, T = draw_case(rng)
        name = "H%d-E%d-k%d-I%d-Is%d-s%d-r%d-g%d-z%s-T%d" % (H, E, k, I, Is, score, renorm, sgate,
                                                          zipf, T)
        shape = wl.small_shape(name, H, E, k, I, Is, score, renorm, sgate)
        w = wl.make_weights(shape, 1000 * seed + n, "cuda", zipf_s=zipf)
        x = wl.make_tokens(shape, T, 2000 * seed + n, "cuda")
        try:
            check_layer_against_oracle(shape, w, x, T, 0)
        except AssertionError as e:
            raise AssertionError("case %d (%s): %s" % (n, name, e)) from e


def test_random_shapes_of_a_few_tokens():
    """One to four tokens: the one-launch kernel (where T * top_k <= 32, else the kernel chain),
    with intermediate sizes that cut the down projection into one to three column chunks."""
    rng = random.Random(14)
    for n in range(160):
        H, E, k, I, Is, score, renorm, sgate, zipf, _ = draw_case(rng)
        T = rng.randint(1, 4)
        if n % 3 == 0:
            I = 32 * rng.choice([65, 100, 136, 150])      # 2080 .. 4800 columns
        if n % 5 == 0 and Is:
            Is = 32 * rng.choice([70, 129, 200])          # 2240 .. 6400 columns
        if E * I * H * 6 > 1_000_000_000:
            continue
        name = "few-H%d-E%d-k%d-I%d-Is%d-s%d-r%d-g%d-z%s-T%d" % (H, E, k, I, Is, score, renorm,
                                                              sgate, zipf, T)
        shape = wl.small_shape(name, H, E, k, I, Is, score, renorm, sgate)
        w = wl.make_weights(shape, 14000 + n, "cuda", zipf_s=zipf)
        x = wl.make_tokens(shape, T, 15000 + n, "cuda")
        try:
            check_layer_against_oracle(shape, w, x, T, 0)
        except AssertionError as e:
            raise AssertionError("case %d (%s): %s" % (n, name, e)) from e

"""The host side of the library on the CPU: the work tables (tiles of the three passes, partial-sum slots, factor
blocks, exchange chunks, second-level sums) that lqsgd_create would build, checked by lqsgd_plan_check for the
benchmark's layer sets, for shapes outside them and for seeded random ones, at several SM counts (the tile sizes
depend on it).  No GPU: nothing here launches or allocates on a device."""
import random

import pytest

from paper_2506_17974_b200 import binding as B
from paper_2506_17974_b200 import workloads as wl

RANKS = (1, 2, 4, 8, 16, 32, 50)


def check(layers, rank, workers, flags=0, sm=148, bits=4, power_iters=0):
    cfg = B.make_config(rank, bits, bits, 127.0, workers, flags=flags, power_iters=power_iters)
    msg = B.plan_check(layers, cfg, sm)
    assert msg == "", (msg, layers, rank, workers, flags, sm)


@pytest.mark.parametrize("sm", [1, 132, 148])
@pytest.mark.parametrize("rank", RANKS)
def test_benchmark_layer_sets(rank, sm):
    check(wl.config1().layers, rank, 1, sm=sm)
    check(wl.config2().layers, rank, 4, sm=sm)
    check(wl.config3().layers, rank, 8, sm=sm)
    check(wl.config5(rank, 4).layers, rank, 16, sm=sm)


@pytest.mark.parametrize("flags", [0, B.FLAG_REGISTER_PATH, B.FLAG_ONE_LAUNCH, B.FLAG_COLUMN_SCALES | B.FLAG_GUARD_WORDS])
@pytest.mark.parametrize("rows,cols", list(wl.CONFIG4_SIZES) + [(50304, 768), (262144, 64), (64, 262144), (4096, 11008),
                                                                (11008, 4096), (16500, 35), (40, 150000), (600, 140000),
                                                                (2, 2), (3, 1000), (1000, 3), (129, 513)])
def test_single_matrices_of_every_family(rows, cols, flags):
    for rank in (2, 8, 16):
        check([(rows, cols)], rank, 1, flags=flags)
    check([(rows, cols)], 4, 3, flags=flags)


def test_bad_arguments_are_refused():
    with pytest.raises(B.LqsgdError):
        B.plan_check([(8, 8)], B.make_config(65, 4, 4, 127.0, 1))
    with pytest.raises(B.LqsgdError):
        B.plan_check([(8, 8)], B.make_config(2, 4, 4, 127.0, 1), sm_count=0)


@pytest.mark.parametrize("kind,expect", [(1, "pass 1"), (2, "pass 2"), (3, "pass 3"), (4, "fold"), (5, "exchange")])
@pytest.mark.parametrize("case", ["resnet_r2", "resnet_r16", "tall_r8", "one_launch"])
def test_planted_defects_are_found(case, kind, expect):
    """The checker is not vacuous: with one tile, one partial-sum slot, one range of workers, one second-level sum
    or one exchange chunk taken out of its private copy of the tables (test support in the C ABI), it names the
    invariant that no longer holds; the undamaged tables pass."""
    layers, rank, workers, flags = {
        "resnet_r2": (wl.config3().layers, 2, 8, 0),
        "resnet_r16": (wl.config5(16, 4).layers, 16, 16, 0),
        "tall_r8": ([(50304, 768), (300, 1)], 8, 2, 0),
        "one_launch": (wl.config2().layers, 4, 4, B.FLAG_ONE_LAUNCH),
    }[case]
    cfg = B.make_config(rank, 4, 4, 127.0, workers, flags=flags)
    assert B.plan_check(layers, cfg) == ""
    B.test_plan_defect(kind)
    msg = B.plan_check(layers, cfg)
    if kind == 4 and case != "tall_r8":
        assert msg == ""                      # no second-level sums in these configurations: nothing to damage
    else:
        assert expect in msg, msg
    assert B.plan_check(layers, cfg) == ""    # the defect armed one call only


def test_seeded_random_layer_sets():
    rng = random.Random(20260617974)
    for case in range(60):
        nl = rng.randint(1, 6)
        layers = []
        for _ in range(nl):
            kind = rng.random()
            if kind < 0.2:
                layers.append((rng.randint(1, 700), 1))                       # a 1-D tensor
            elif kind < 0.5:
                layers.append((rng.randint(2, 600), rng.randint(2, 5000)))
            elif kind < 0.7:
                layers.append((rng.randint(2, 40000), rng.randint(2, 300)))   # tall
            elif kind < 0.9:
                layers.append((rng.randint(2, 300), rng.randint(2, 200000)))  # wide
            else:
                layers.append((4 * rng.randint(1, 800), 4 * rng.randint(1, 800)))
        if not any(n > 1 and m > 1 for n, m in layers):
            layers.append((7, 9))
        rank = rng.choice((1, 2, 3, 5, 8, 12, 16, 30, 64))
        workers = rng.choice((1, 2, 3, 4, 8, 16))
        flags = rng.choice((0, 0, B.FLAG_REGISTER_PATH, B.FLAG_ONE_LAUNCH, B.FLAG_QUANTIZE_VECTORS, B.FLAG_AVERAGE_VALUES))
        sm = rng.choice((1, 16, 108, 132, 148, 160))
        check(layers, rank, workers, flags=flags, sm=sm, power_iters=rng.choice((0, 0, 2)))

"""Host-side checks of the weight streaming layout and the work partition (no GPU needed).

The library walks every thread block's share of an operation the way the kernel's weight streamer
and tensor-core thread do (pass by pass, stage by stage, through the addresses the shared-memory
descriptors generate) and checks that every 16-byte unit of the matrix is met exactly once, at the
offset the packing step writes it to."""
import numpy as np
import pytest

from sdv_inputs import get_config
from paper_2510_15312_b200.binding import EINVAL, OK, config_from, layout_check, plan

CONFIGS = ["tiny", "mini_gqa", "mini_hd128", "qwen0.5b", "qwen1.5b", "llama3b", "qwen7b"]


@pytest.mark.parametrize("name", CONFIGS)
def test_partitions_of_every_configuration_cover_each_matrix_once(name):
    cfg = get_config(name)
    for blocks in (148, 132, 7):
        ops, sp = plan(config_from(cfg, k_max=16), blocks, cfg.k + 1)
        if blocks > 100:
            assert sp[5] == 1 and sp[2] >= 2, (name, blocks, sp)      # the plan fits, at least two ring slots
        gu = ops[2]
        for i, o in enumerate(ops):
            assert layout_check(o, gu, blocks) == OK, (name, blocks, i, o)
        # gate|up and down share one split of the SwiGLU columns
        assert ops[3][7] == 1 and ops[3][1] == gu[0] // gu[6]


def test_random_partitions_and_ragged_shapes():
    rng = np.random.default_rng(0)
    for _ in range(300):
        RW = int(rng.choice([1, 2, 4, 8, 16]))
        SK = int(rng.integers(1, 64 // RW + 1))
        unit = int(rng.choice([1, 2]))
        T = unit * int(rng.integers(1, 40))
        K16 = int(rng.integers(1, 50))
        G = int(rng.integers(1, 20))
        P_row = int(rng.integers(1, min(G, T // unit) + 1))
        P_k = int(rng.integers(1, min(G // P_row, K16) + 1))
        o = [T, K16, P_row, P_k, RW, SK, unit, 0]
        assert layout_check(o, o, G) == OK, o
    # a follower takes the columns its gate|up partition produces
    for _ in range(100):
        G = int(rng.integers(1, 20))
        units = int(rng.integers(1, 60))
        gu = [2 * units, int(rng.integers(1, 20)), min(G, units), 1, 16, 4, 2, 0]
        down = [int(rng.integers(1, 30)), units, 1, gu[2], 16, int(rng.integers(1, 5)), 1, 1]
        assert layout_check(gu, gu, G) == OK
        assert layout_check(down, gu, G) == OK, (down, gu)


def test_malformed_descriptions_are_rejected():
    good = [16, 8, 2, 2, 8, 8, 1, 0]
    assert layout_check(good, good, 8) == OK
    for bad in ([0, 8, 1, 1, 8, 8, 1, 0], [16, 8, 1, 1, 8, 9, 1, 0], [15, 8, 1, 1, 8, 8, 2, 0]):
        assert layout_check(bad, good, 8) == EINVAL

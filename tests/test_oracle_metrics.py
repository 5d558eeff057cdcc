"""Pins of the two error yardsticks every parity assert goes through, against values worked out by hand.
CPU only."""
import numpy as np

from oracle import ab_oracle as orc


def test_rel_frob_hand_values():
    a = np.array([[3.0, 0.0], [0.0, 0.0]])
    b = np.array([[0.0, 0.0], [0.0, 4.0]])
    # a - b = [[3, 0], [0, -4]]: norm 5; ||b|| = 4
    assert orc.rel_frob(a, b) == 1.25
    assert orc.rel_frob(b, b) == 0.0
    assert orc.rel_frob(np.zeros((2, 2)), np.zeros((2, 2))) == 0.0
    # not symmetric: the second argument is the yardstick
    assert np.isclose(orc.rel_frob(b, a), 5.0 / 3.0)
    # float32 inputs are widened, not compared in float32
    assert orc.rel_frob(np.float32([1.0 + 2.0 ** -20]), np.float32([1.0])) == 2.0 ** -20


def test_max_tile_rel_frob_finds_one_bad_tile():
    rng = np.random.default_rng(0)
    b = rng.standard_normal((300, 200))
    a = b.copy()
    assert orc.max_tile_rel_frob(a, b) == 0.0
    # one 128 x 64 tile replaced by zeros: the whole-matrix figure stays small, the tile figure is 1
    a[128:256, 64:128] = 0.0
    whole = orc.rel_frob(a, b)
    assert whole < 0.4
    assert np.isclose(orc.max_tile_rel_frob(a, b), 1.0)
    # hand value on a 2 x 2 grid of 1 x 1 tiles
    b2 = np.array([[1.0, 2.0], [4.0, 8.0]])
    a2 = np.array([[1.5, 2.0], [4.0, 9.0]])
    assert orc.max_tile_rel_frob(a2, b2, 1, 1) == 0.5
    # ragged edge tiles are covered
    a3 = b.copy()
    a3[299, 199] += 1.0
    edge = b[256:300, 192:200]
    assert np.isclose(orc.max_tile_rel_frob(a3, b), 1.0 / np.linalg.norm(edge))
    # a tile of zeros in the reference does not divide by zero
    b4 = b.copy()
    b4[0:128, 0:64] = 0.0
    a4 = b4.copy()
    a4[0, 0] = 1e-9
    assert np.isfinite(orc.max_tile_rel_frob(a4, b4))

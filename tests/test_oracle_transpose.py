"""Pins for the transpose oracle: a hand example, the loop definition, and involution."""

import numpy as np

from oracle import transpose as T


def test_hand_example():
    x = np.array([[1, 2, 3], [4, 5, 6]], dtype=np.uint16)
    want = np.array([[1, 4], [2, 5], [3, 6]], dtype=np.uint16)
    assert np.array_equal(T.transpose_loops(x), want) and np.array_equal(T.transpose(x), want)


def test_library_path_matches_the_definition_and_is_an_involution():
    rng = np.random.default_rng(0)
    for (M, N) in [(1, 1), (7, 13), (64, 64), (65, 130)]:
        x = rng.integers(0, 65536, size=(M, N)).astype(np.uint16)
        assert np.array_equal(T.transpose(x), T.transpose_loops(x))
        assert np.array_equal(T.transpose(T.transpose(x)), x)
        assert T.transpose(x).flags["C_CONTIGUOUS"]

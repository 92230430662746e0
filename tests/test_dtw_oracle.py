"""Pins for the DTW oracle: closed forms, brute force over all monotone paths, path validity."""
import itertools

import numpy as np

from oracle import dtw_oracle as D
from paper_2412_11272_b200 import inputs as I


def _valid(path, N, M):
    assert path[0] == (0, 0) and path[-1] == (N - 1, M - 1)
    for (a, b), (c, d) in zip(path, path[1:]):
        assert (c - a, d - b) in ((1, 1), (1, 0), (0, 1))


def test_zero_diagonal_is_followed():
    C = np.ones((6, 6), np.float32) - np.eye(6, dtype=np.float32)
    total, path, start = D.dtw(C)
    assert total == 0.0 and path == [(i, i) for i in range(6)] and list(start) == list(range(6))


def test_single_row_and_single_column():
    C = np.arange(1, 8, dtype=np.float32).reshape(1, 7)
    total, path, start = D.dtw(C)
    assert total == 28.0 and path == [(0, j) for j in range(7)] and list(start) == [0]
    total, path, start = D.dtw(C.T)
    assert total == 28.0 and path == [(i, 0) for i in range(7)] and list(start) == [0] * 7


def test_zero_cost_bands_give_their_first_frames():
    bounds = [0, 3, 4, 9, 12]
    C = np.ones((4, 12), np.float32)
    for i in range(4):
        C[i, bounds[i]:bounds[i + 1]] = 0.0
    total, path, start = D.dtw(C)
    assert total == 0.0 and list(start) == bounds[:4]
    _valid(path, 4, 12)


def _all_paths(N, M):
    def rec(i, j):
        if (i, j) == (N - 1, M - 1):
            yield [(i, j)]
            return
        for di, dj in ((1, 1), (1, 0), (0, 1)):
            if i + di < N and j + dj < M:
                for rest in rec(i + di, j + dj):
                    yield [(i, j)] + rest
    return rec(0, 0)


def test_brute_force_over_all_monotone_paths():
    rng = np.random.default_rng(3)
    for N, M in ((3, 4), (4, 4), (2, 6), (5, 3)):
        C = rng.random((N, M)).astype(np.float32)
        total, path, _ = D.dtw(C)
        _valid(path, N, M)
        best = min(float(np.sum([np.float64(C[a, b]) for a, b in p])) for p in _all_paths(N, M))
        assert abs(float(total) - best) < 1e-5
        assert abs(sum(float(C[a, b]) for a, b in path) - best) < 1e-5


def test_synthetic_attention_costs_recover_a_monotone_alignment():
    C = I.dtw_cost(1, 0, 40, 300)
    total, path, start = D.dtw(C)
    _valid(path, 40, 300)
    assert np.all(np.diff(start) >= 0) and start[0] == 0
    centres = np.argmin(C - 0 * C, axis=1)
    assert np.mean(np.abs(start - centres)) < 30            # starts sit near (before) the band centres


def test_tie_order_on_hand_worked_matrices():
    """The stated tie order (diagonal, then the step in the token index, then the step in the frame
    index), on matrices small enough to fill in by hand.
    All ones, 2 x 3: D = [[1, 2, 3], [2, 2, 3]].  The last cell sees diagonal D[0,1] = 2 and left
    D[1,1] = 2 (up is 3): the tie goes to the diagonal, so the path is (0,0) (0,1) (1,2) and token 1
    starts at frame 2 (a left-first rule would give (0,0) (1,1) (1,2) and frame 1)."""
    total, path, start = D.dtw(np.ones((2, 3), np.float32))
    assert total == 3.0 and path == [(0, 0), (0, 1), (1, 2)] and list(start) == [0, 2]
    # C = [[5, -1], [-1, 0]]: D = [[5, 4], [4, 4]]; the last cell sees diagonal 5, up 4, left 4: the tie
    # between the two steps goes to the step in the token index, i.e. the predecessor (0, 1)
    total, path, start = D.dtw(np.array([[5, -1], [-1, 0]], np.float32))
    assert total == 4.0 and path == [(0, 0), (0, 1), (1, 1)] and list(start) == [0, 1]
    # all zeros, 3 x 3: everything ties, the diagonal wins at every cell
    total, path, start = D.dtw(np.zeros((3, 3), np.float32))
    assert total == 0.0 and path == [(0, 0), (1, 1), (2, 2)] and list(start) == [0, 1, 2]

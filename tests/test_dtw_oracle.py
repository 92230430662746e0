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

"""Dynamic time warping of a token-by-frame cost matrix.  TEST INFRASTRUCTURE ONLY.

The paper (Sec. 3.2 "Workload mapping", Sec. 4.3.2) estimates token timestamps with DTW over the
decoder's cross-attention and cites the classic dynamic-programming formulation; it gives no
further detail, so this is the textbook definition:

    D[0, 0] = C[0, 0]
    D[i, j] = C[i, j] + min(D[i-1, j-1], D[i-1, j], D[i, j-1])        (missing neighbours = +inf)

and the path is traced back from (N-1, M-1) to (0, 0) through the arg-min predecessors.  The
accumulation runs in float32 in exactly this order, and ties prefer the diagonal, then the step
in i, then the step in j, so that a float32 implementation can be compared bit for bit (the
arg-min is an integer decided by floating point: both sides decide in the same precision).
`token_start[i]` is the first frame of token i on the path.
"""
from __future__ import annotations

import numpy as np


def dtw(cost):
    C = np.asarray(cost, dtype=np.float32)
    N, M = C.shape
    inf = np.float32(np.inf)
    D = np.full((N, M), inf, dtype=np.float32)
    step = np.zeros((N, M), dtype=np.uint8)          # 0 diagonal, 1 from (i-1, j), 2 from (i, j-1)
    for i in range(N):
        for j in range(M):
            if i == 0 and j == 0:
                D[0, 0] = C[0, 0]
                continue
            best, s = (D[i - 1, j - 1] if i > 0 and j > 0 else inf), 0
            up = D[i - 1, j] if i > 0 else inf
            left = D[i, j - 1] if j > 0 else inf
            if up < best:
                best, s = up, 1
            if left < best:
                best, s = left, 2
            D[i, j] = np.float32(C[i, j] + best)
            step[i, j] = s
    i, j = N - 1, M - 1
    path = [(i, j)]
    while (i, j) != (0, 0):
        s = step[i, j]
        if s == 0:
            i, j = i - 1, j - 1
        elif s == 1:
            i -= 1
        else:
            j -= 1
        path.append((i, j))
    path.reverse()
    token_start = np.full(N, -1, dtype=np.int32)
    for (a, b) in path:
        if token_start[a] < 0:
            token_start[a] = b
    return D[N - 1, M - 1], path, token_start

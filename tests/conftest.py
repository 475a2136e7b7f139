import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def read_golden(name):
    """Parse tests/golden/<name>: '#' comments, 'case <id>' headers, 'key: v v v' lines."""
    cases, cur = {}, None
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            if line.startswith("case "):
                cur = {}
                cases[line[5:].strip()] = cur
                continue
            key, _, rest = line.partition(":")
            cur[key.strip()] = [int(t) for t in rest.split()]
    return cases


@pytest.fixture(scope="session")
def golden():
    return read_golden


def lane_tile_rows(M, S, R, C):
    """Row of W behind (tile t = 32*s + L, local row i) for the LANE_TILE row map, written out from its
    definition in the public header; -1 where that row does not exist.  Shape (32*S, R)."""
    import numpy as np
    t = np.arange(32 * S)[:, None]
    i = np.arange(R)[None, :]
    s, L = t // 32, t % 32
    rows = (((i // C) * S + s) * C + i % C) * 32 + L
    return np.where(rows < M, rows, -1)


def permute_for_lane_tiles(W, mask, S, R, C):
    """(W', mask', rows): the matrix whose consecutive tiles of R rows are the library's lane tiles, so
    that the oracle's encoder with tile_rows=R sees what the library stores; rows[p] = row of W at p."""
    import numpy as np
    M, K = W.shape
    rows = lane_tile_rows(M, S, R, C).reshape(-1)
    live = rows >= 0
    assert np.array_equal(np.sort(rows[live]), np.arange(M))         # a permutation of the rows
    if mask is None:
        mask = ((W.view(np.uint16) & 0x7FFF) != 0).astype(np.uint8)
    Wp = np.zeros((rows.size, K), W.dtype)
    mp = np.zeros((rows.size, K), np.uint8)
    Wp[live] = W[rows[live]]
    mp[live] = mask[rows[live]]
    return Wp, mp, rows

"""Host logic of the CUDA library: the cell table that prunes the nearest-grid-point search must
never exclude the true nearest point (Section 2: pairs go to the nearest of n fixed points).  Checked
without a GPU against brute force in float64 on Gaussian points, on points hugging cell borders and
on points hugging Voronoi edges."""
import numpy as np
import pytest

from paper_2501_19392_b200 import synth


def _candidates(table, lists, cells, half, y):
    """Candidate lists (8 wide, ascending, padded by repetition) of the cells the points fall in; `brute`
    marks cells that say "search all points", `second` those that refer to a second-level list."""
    w = 2.0 * half / cells
    ix = np.clip(np.floor((y[:, 0] + half) / w).astype(np.int64), 0, cells - 1)   # the kernel's cell index saturates
    iy = np.clip(np.floor((y[:, 1] + half) / w).astype(np.int64), 0, cells - 1)
    e = table[iy, ix].astype(np.int64)
    brute = e == 0xFFFFFFFF
    second = (e >= 0xFF000000) & ~brute
    first = np.stack([(e >> 24) & 0xFF, (e >> 16) & 0xFF, (e >> 8) & 0xFF, e & 0xFF], axis=1)
    cand = np.concatenate([first, first[:, 3:4].repeat(4, axis=1)], axis=1)
    if second.any():
        cand[second] = lists[e[second] & 0xFFFFFF].astype(np.int64)
    return cand, brute, second


@pytest.mark.parametrize("n", [16, 64, 256])
def test_table_keeps_the_nearest_point(n):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(n, seed=7, n_samples=1 << 14, iters=25)
    cells, half, table, lists = api.search_table(grid)
    assert len(lists) <= api.SEARCH_TABLE_LIST_WORDS // 2
    assert cells == 64 and half >= np.abs(grid).max() + 2.0
    G = grid.astype(np.float64)
    rng = np.random.default_rng(n)
    w = 2.0 * half / cells
    gauss = rng.standard_normal((200000, 2))
    # points within 1e-6 cells of a cell border (both sides)
    border = (rng.integers(-cells // 2, cells // 2, size=(50000, 2)) * w
              + rng.choice([-1e-6, 1e-6], size=(50000, 2)) * w)
    border[:, 1] = rng.standard_normal(50000)
    # points on the perpendicular bisector of two neighbouring grid points, nudged to either side
    i = rng.integers(0, n, 50000)
    d2 = ((G[i][:, None, :] - G[None, :, :]) ** 2).sum(-1)
    d2[np.arange(50000), i] = np.inf
    j = d2.argmin(1)
    mid = 0.5 * (G[i] + G[j])
    dirn = G[j] - G[i]
    perp = np.stack([-dirn[:, 1], dirn[:, 0]], 1)
    edge = mid + perp * rng.uniform(-0.5, 0.5, (50000, 1)) + dirn * rng.choice([-1e-5, 1e-5], (50000, 1))
    for name, y in (("gauss", gauss), ("border", border), ("edge", edge)):
        dist = ((y[:, None, :] - G[None, :, :]) ** 2).sum(-1)
        order = np.argsort(dist, axis=1)
        best = order[:, 0]
        margin = (np.take_along_axis(dist, order[:, 1:2], 1)[:, 0] - dist[np.arange(len(y)), best])
        cand, brute, lvl2 = _candidates(table, lists, cells, half, y)
        listed = (cand == best[:, None]).any(axis=1)
        assert np.all(listed | brute), "%s: nearest point missing from %d cells" % (name, (~(listed | brute)).sum())
        # near-ties (fp32 could pick either point): both contenders must be listed
        tie = (margin < 1e-5) & ~brute
        second = order[:, 1]
        assert np.all((cand[tie] == second[tie][:, None]).any(axis=1))
        # candidates are ascending so that the first minimum is the lowest index
        asc = ~brute
        assert np.all(np.diff(cand[asc], axis=1) >= 0)
        # the kernel's fast path evaluates three candidates for n = 16 and four otherwise: cells with
        # more must go through a second-level list
        plain = ~brute & ~lvl2
        distinct = (np.diff(cand[plain][:, :4], axis=1) > 0).sum(axis=1) + 1
        assert np.all(distinct <= (3 if n == 16 else 4))
        if n == 16:     # the fourth byte only repeats the third
            assert np.all(cand[plain][:, 3] == cand[plain][:, 2])
        if lvl2.any():
            assert np.all((np.diff(cand[lvl2], axis=1) > 0).sum(axis=1) + 1 > (3 if n == 16 else 4))
        # values outside the square land in border cells, which must all say "search all points"
        assert np.all(table[0, :] == 0xFFFFFFFF) and np.all(table[-1, :] == 0xFFFFFFFF)
        assert np.all(table[:, 0] == 0xFFFFFFFF) and np.all(table[:, -1] == 0xFFFFFFFF)
        if n <= 64:             # second-level lists exist only for the 256-point grid
            assert not lvl2.any() and len(lists) == 0
        if name == "gauss":     # the exhaustive search must stay rare
            assert brute.mean() < (0.02 if n <= 64 else 1e-3), brute.mean()
            assert lvl2.mean() < 0.25, lvl2.mean()

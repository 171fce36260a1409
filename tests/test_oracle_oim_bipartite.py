"""Pins for the oracle's full-line (bipartite) reading of OIM's matching (Section 3.2): every
even cell of a line is compared with every odd cell of that line.  CPU only."""
import itertools

import numpy as np
import pytest


def _rand_grid(B, H, W, D, seed):
    return np.random.default_rng(seed).standard_normal((B, H, W, D)).astype(np.float32)


def _cos(a, b):
    na, nb = np.linalg.norm(a), np.linalg.norm(b)
    return 0.0 if na == 0 or nb == 0 else float(a @ b / (na * nb))


@pytest.mark.parametrize("H,W,target,D", [(6, 6, 9, 16), (8, 5, 10, 8), (7, 9, 21, 12), (12, 12, 16, 32), (3, 3, 1, 4)])
def test_invariants(oracle_mod, H, W, target, D):
    x = _rand_grid(2, H, W, D, seed=H * 100 + W + 7)
    r = oracle_mod.oim(x, target=target, matching="bipartite")
    Hf, Wf = r["grid"]
    assert Hf * Wf == target
    xs = x.reshape(2, H * W, D).astype(np.float64)
    for b in range(2):
        m, s, t = r["map"][b], r["sizes"][b], r["tokens"][b]
        assert m.min() >= 0 and m.max() < target
        assert s.sum() == H * W
        assert np.array_equal(np.bincount(m, minlength=target), s)
        ref = np.stack([xs[b][m == c].mean(0) for c in range(target)])
        np.testing.assert_allclose(t, ref, rtol=1e-12, atol=1e-12)


def test_lines_of_two_or_three_cells_equal_the_adjacent_reading(oracle_mod):
    # with at most three cells in a line every odd cell IS a neighbour of every even cell,
    # so the two readings must give the same result (the adjacent one is pinned on its own)
    for (H, W, hw) in [(3, 3, (1, 1)), (2, 3, (1, 2)), (3, 2, (2, 1)), (3, 3, (2, 2))]:
        x = _rand_grid(2, H, W, 6, seed=H * 10 + W)
        a = oracle_mod.oim(x, out_hw=hw, r=1)
        b = oracle_mod.oim(x, out_hw=hw, r=1, matching="bipartite")
        # after the first shrink of an axis its lines have at most two cells left, still covered
        np.testing.assert_array_equal(a["map"], b["map"])
        np.testing.assert_allclose(a["tokens"], b["tokens"], rtol=0, atol=1e-13)


def test_a_distant_twin_is_found_where_the_adjacent_reading_cannot(oracle_mod):
    # one row of 8 mutually orthogonal cells, except that cell 0 equals cell 5 and cell 6 is
    # close to cell 1: the full-line matching must merge 0 -> 5 and 6 -> 1
    x = np.zeros((1, 1, 8, 8), np.float32)
    for j in range(8):
        x[0, 0, j, j] = 1.0 + j
    x[0, 0, 0] = 3.0 * x[0, 0, 5]                      # cosine 1 with cell 5
    x[0, 0, 6] = x[0, 0, 1] + 0.25 * x[0, 0, 6]        # cosine ~0.75 with cell 1
    r = oracle_mod.oim(x, out_hw=(1, 6), matching="bipartite")
    assert r["trace"][0].tolist() == [(0 << 16) | 5, (6 << 16) | 1]
    # survivors in order: 1(+6), 2, 3, 4, 5(+0), 7
    assert r["map"][0].tolist() == [4, 0, 1, 2, 3, 4, 0, 5]
    assert r["sizes"][0].tolist() == [2, 1, 1, 1, 2, 1]
    np.testing.assert_allclose(r["tokens"][0][4], (x[0, 0, 5].astype(np.float64) + x[0, 0, 0]) / 2, atol=1e-13)
    np.testing.assert_allclose(r["tokens"][0][0], (x[0, 0, 1].astype(np.float64) + x[0, 0, 6]) / 2, atol=1e-13)
    # the adjacent reading sees only orthogonal neighbours for cell 0
    adj = oracle_mod.oim(x, out_hw=(1, 6))
    assert adj["map"][0].tolist() != r["map"][0].tolist()


def test_constant_line_ties_go_to_the_lowest_positions(oracle_mod):
    x = np.ones((1, 1, 7, 4), np.float32)
    r = oracle_mod.oim(x, out_hw=(1, 5), matching="bipartite")
    # A cells 0 and 2 (lowest positions) both propose B cell 1 (lowest position)
    assert r["trace"][0].tolist() == [(0 << 16) | 1, (2 << 16) | 1]
    assert r["sizes"][0].tolist() == [3, 1, 1, 1, 1]
    assert r["map"][0].tolist() == [0, 0, 0, 1, 2, 3, 4]


def test_several_sources_may_share_one_destination_and_weights_are_sizes(oracle_mod):
    # second width step: a size-3 cell (from the first step) absorbs another; the result must be
    # the plain mean of all four sources, i.e. the merge is size-weighted
    x = _rand_grid(1, 1, 9, 5, seed=2) * 0.05
    base = np.arange(1, 6, dtype=np.float32)
    for j in (0, 1, 2, 6):
        x[0, 0, j] += base                      # cells 0, 1, 2, 6 are near-parallel
    r = oracle_mod.oim(x, out_hw=(1, 5), matching="bipartite")
    c = r["map"][0][1]
    assert [r["map"][0][j] for j in (0, 1, 2, 6)] == [c] * 4
    assert r["sizes"][0][c] == 4
    np.testing.assert_allclose(r["tokens"][0][c], x[0, 0, [0, 1, 2, 6]].astype(np.float64).mean(0), atol=1e-13)


def test_width_step_equals_height_step_on_the_transposed_grid(oracle_mod):
    x = _rand_grid(1, 6, 7, 10, seed=13)
    a = oracle_mod.oim(x, out_hw=(3, 4), matching="bipartite")
    b = oracle_mod.oim(np.ascontiguousarray(x.transpose(0, 2, 1, 3)), out_hw=(4, 3), height_first=True,
                       matching="bipartite")
    ta = a["tokens"][0].reshape(3, 4, 10)
    tb = b["tokens"][0].reshape(4, 3, 10).transpose(1, 0, 2)
    np.testing.assert_allclose(ta, tb, rtol=0, atol=1e-13)


def _brute_force_step(grid, sizes, axis, m):
    """Every way to pick m even-position cells of a line and ANY odd-position cell of the line for
    each of them; the plan with the largest total cosine wins (lines are independent)."""
    h, w, D = grid.shape
    if axis == 1:
        g, s = _brute_force_step(grid.transpose(1, 0, 2), sizes.T, 0, m)
        return g.transpose(1, 0, 2), s.T
    new = np.zeros((h, w - m, D))
    news = np.zeros((h, w - m), np.int64)
    evens, odds = list(range(0, w, 2)), list(range(1, w, 2))
    for r in range(h):
        best, best_plan = -np.inf, None
        for subset in itertools.combinations(evens, m):
            for dsts in itertools.product(odds, repeat=m):
                tot = sum(_cos(grid[r, a], grid[r, d]) for a, d in zip(subset, dsts))
                if tot > best + 1e-15:
                    best, best_plan = tot, list(zip(subset, dsts))
        vec = {j: sizes[r, j] * grid[r, j] for j in range(w)}
        sz = {j: sizes[r, j] for j in range(w)}
        for a, d in best_plan:
            vec[d] = vec[d] + sizes[r, a] * grid[r, a]
            sz[d] += sizes[r, a]
        keep = [j for j in range(w) if j not in {a for a, _ in best_plan}]
        for o, j in enumerate(keep):
            new[r, o] = vec[j] / sz[j]
            news[r, o] = sz[j]
    return new, news


@pytest.mark.parametrize("H,W,Hf,Wf", [(4, 6, 2, 4), (5, 5, 3, 3), (6, 4, 3, 2), (2, 7, 1, 3), (5, 6, 4, 2)])
def test_plan_maximises_total_similarity_on_tiny_grids(oracle_mod, H, W, Hf, Wf):
    for seed in range(4):
        x = _rand_grid(1, H, W, 5, seed=seed + 40)
        r = oracle_mod.oim(x, out_hw=(Hf, Wf), matching="bipartite")
        grid = x[0].astype(np.float64)
        sizes = np.ones((H, W), np.int64)
        for axis, m in oracle_mod.oim_schedule(H, W, Hf, Wf):
            grid, sizes = _brute_force_step(grid, sizes, axis, m)
        np.testing.assert_allclose(r["tokens"][0].reshape(Hf, Wf, 5), grid, rtol=1e-12, atol=1e-12)
        assert np.array_equal(r["sizes"][0].reshape(Hf, Wf), sizes)


def test_replay_accepts_own_trace_and_flags_a_wrong_one(oracle_mod):
    x = _rand_grid(2, 6, 6, 8, seed=19)
    run = oracle_mod.oim(x, target=9, matching="bipartite")
    assert np.all(run["stats"][:, 0] > 1e-6)
    again = oracle_mod.oim(x, target=9, trace=run["trace"], matching="bipartite")
    assert np.all(again["stats"][:, 2:] == 0)
    np.testing.assert_array_equal(again["map"], run["map"])
    np.testing.assert_array_equal(again["tokens"], run["tokens"])
    bad = run["trace"].copy()
    a, b = bad[0][0] >> 16, bad[0][0] & 0xffff
    bad[0][0] = (a << 16) | (b + 2 if b + 2 < 6 else b - 2)     # another odd cell of the line
    flagged = oracle_mod.oim(x, target=9, trace=bad, tol=1e-9, matching="bipartite")
    assert flagged["stats"][0, 2] > 0
    malformed = run["trace"].copy()
    malformed[0][0] = (1 << 16) | 1                                # an odd source
    assert oracle_mod.oim(x, target=9, trace=malformed, matching="bipartite")["stats"][0, 2] > 0


def test_replay_selection_rule_on_a_line_with_known_margins(oracle_mod):
    # one line of 2-D unit vectors at angles 0, 0.1, 0.5, 0.8, 1.5, 2.0, 3.0: an even cell's proposal
    # over ALL odd cells.  cell 0 -> cell 1 (cos 0.1);  cell 2 -> cell 3 (cos 0.3; cell 1: cos 0.4);
    # cell 4 -> cell 5 (cos 0.5; cell 3: cos 0.7);  cell 6 -> cell 5 (cos 1.0)
    a = np.array([0.0, 0.1, 0.5, 0.8, 1.5, 2.0, 3.0])
    x = np.stack([np.cos(a), np.sin(a)], axis=-1).astype(np.float32)[None, None]
    own = oracle_mod.oim(x, out_hw=(1, 6), matching="bipartite")
    assert own["trace"][0].tolist() == [(0 << 16) | 1]
    margin = 0.9950041652780258 - 0.955336489125606           # cos 0.1 - cos 0.3
    np.testing.assert_allclose(own["stats"][0, 0], margin, atol=1e-6)
    swapped = np.array([[(2 << 16) | 3]], np.int32)            # merges cell 2 although cell 0 scores higher
    strict = oracle_mod.oim(x, out_hw=(1, 6), trace=swapped, tol=margin - 1e-3, matching="bipartite")
    assert strict["stats"][0, 2] > 0
    lenient = oracle_mod.oim(x, out_hw=(1, 6), trace=swapped, tol=margin + 1e-3, matching="bipartite")
    assert lenient["stats"][0, 2] == 0 and lenient["stats"][0, 3] > 0
    assert lenient["map"][0].tolist() == [0, 1, 2, 2, 3, 4, 5]
    # two merges: {0, 4} instead of {0, 2}, margin cos 0.3 - cos 0.5
    swapped2 = np.array([[(0 << 16) | 1, (4 << 16) | 5]], np.int32)
    margin2 = 0.955336489125606 - 0.8775825618903728
    assert oracle_mod.oim(x, out_hw=(1, 5), trace=swapped2, tol=margin2 - 1e-3, matching="bipartite")["stats"][0, 2] > 0
    assert oracle_mod.oim(x, out_hw=(1, 5), trace=swapped2, tol=margin2 + 1e-3, matching="bipartite")["stats"][0, 2] == 0
    # a proposal that is not the cell's best one: cell 2 into cell 1 (cos 0.4) instead of cell 3 (cos 0.3)?
    # cos 0.4 = 0.92106 < cos 0.3: 0.03428 below the best, so it is a violation below that and accepted above
    worse = np.array([[(0 << 16) | 1, (2 << 16) | 1]], np.int32)
    gap = 0.955336489125606 - 0.9210609940028851
    assert oracle_mod.oim(x, out_hw=(1, 5), trace=worse, tol=gap - 1e-3, matching="bipartite")["stats"][0, 2] > 0
    assert oracle_mod.oim(x, out_hw=(1, 5), trace=worse, tol=gap + 1e-3, matching="bipartite")["stats"][0, 2] == 0

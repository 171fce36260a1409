"""Pins for the OIM oracle: invariants the paper fixes, special cases with a textbook
answer, and brute-force enumeration of merge plans on tiny grids (CPU only)."""
import itertools
import os

import numpy as np
import pytest

import luvc_inputs as gi

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_grid(B, H, W, D, seed):
    return np.random.default_rng(seed).standard_normal((B, H, W, D)).astype(np.float32)


def _cos(a, b):
    na, nb = np.linalg.norm(a), np.linalg.norm(b)
    return 0.0 if na == 0 or nb == 0 else float(a @ b / (na * nb))


# ------------------------------------------------------------------ schedule / target grid


def test_final_grid_and_step_count_match_the_configurations(oracle_mod):
    for line in open(os.path.join(GOLDEN, "oim_schedules.txt")):
        if line.startswith("#") or not line.strip():
            continue
        H, W, target, Hf, Wf, steps = map(int, line.split())
        assert oracle_mod.oim_final_dims(H, W, target) == (Hf, Wf)
        sched = oracle_mod.oim_schedule(H, W, Hf, Wf)
        assert len(sched) == steps
        assert sum(m for a, m in sched if a == 0) == W - Wf
        assert sum(m for a, m in sched if a == 1) == H - Hf
        assert all(1 <= m <= 2 for _, m in sched)
        # width first, then strict alternation while both axes still shrink
        assert sched[0][0] == 0
        both = min(sum(1 for a, _ in sched if a == 0), sum(1 for a, _ in sched if a == 1))
        assert [a for a, _ in sched[: 2 * both]] == [0, 1] * both


def test_final_grid_rule(oracle_mod):
    # closest aspect ratio in log scale, tie to the larger height
    assert oracle_mod.oim_final_dims(6, 6, 8) == (4, 2)
    assert oracle_mod.oim_final_dims(4, 8, 8) == (2, 4)
    assert oracle_mod.oim_final_dims(5, 7, 35) == (5, 7)
    with pytest.raises(ValueError):
        oracle_mod.oim_final_dims(4, 4, 7)      # 7 = 1x7 or 7x1: neither fits in 4x4
    with pytest.raises(ValueError):
        oracle_mod.oim_final_dims(4, 4, 17)
    assert oracle_mod.oim_schedule(5, 5, 5, 5) == []
    assert oracle_mod.oim_schedule(3, 3, 3, 1) == [(0, 2)]
    assert oracle_mod.oim_schedule(2, 2, 1, 1) == [(0, 1), (1, 1)]
    assert oracle_mod.oim_schedule(2, 2, 1, 1, height_first=True) == [(1, 1), (0, 1)]


# ------------------------------------------------------------------ invariants


@pytest.mark.parametrize("H,W,target,D", [(6, 6, 9, 16), (8, 5, 10, 8), (7, 9, 21, 12), (12, 12, 16, 32), (3, 3, 1, 4)])
def test_invariants(oracle_mod, H, W, target, D):
    x = _rand_grid(3, H, W, D, seed=H * 100 + W)
    r = oracle_mod.oim(x, target=target)
    Hf, Wf = r["grid"]
    assert Hf * Wf == target
    xs = x.reshape(3, H * W, D).astype(np.float64)
    for b in range(3):
        m, s, t = r["map"][b], r["sizes"][b], r["tokens"][b]
        assert m.min() >= 0 and m.max() < target
        assert s.sum() == H * W
        assert np.array_equal(np.bincount(m, minlength=target), s)
        # a merged token is the plain mean of its sources (size-weighted means compose to it)
        ref = np.stack([xs[b][m == c].mean(0) for c in range(target)])
        np.testing.assert_allclose(t, ref, rtol=1e-12, atol=1e-12)
        # order: a source at (h, w) ends in a cell (hf, wf) that is not below/right of it and
        # is displaced by no more than the rows / columns removed
        hh, ww = np.divmod(np.arange(H * W), W)
        hf, wf = np.divmod(m, Wf)
        assert np.all(hf <= hh) and np.all(hf >= hh - (H - Hf))
        assert np.all(wf <= ww) and np.all(wf >= ww - (W - Wf))


def test_row_major_order_is_preserved_inside_every_line(oracle_mod):
    # one width step: surviving cells keep their left-to-right order in every row
    x = _rand_grid(1, 5, 9, 8, seed=3)
    r = oracle_mod.oim(x, out_hw=(5, 7))
    m = r["map"][0].reshape(5, 9)
    for h in range(5):
        cells = m[h]
        assert np.all(cells // 7 == h)               # a width step never moves a token to another row
        assert np.all(np.diff(cells % 7) >= 0)       # order along the row kept


def test_identity_when_target_is_the_input_size(oracle_mod):
    x = _rand_grid(2, 4, 6, 8, seed=1)
    r = oracle_mod.oim(x, target=24)
    assert r["grid"] == (4, 6)
    np.testing.assert_array_equal(r["tokens"], x.reshape(2, 24, 8).astype(np.float64))
    assert np.all(r["sizes"] == 1)
    assert np.array_equal(r["map"][0], np.arange(24))


def test_batch_independence(oracle_mod):
    x = _rand_grid(4, 6, 6, 8, seed=5)
    full = oracle_mod.oim(x, target=9)
    for b in range(4):
        one = oracle_mod.oim(x[b:b + 1], target=9)
        np.testing.assert_array_equal(one["map"][0], full["map"][b])
        np.testing.assert_array_equal(one["tokens"][0], full["tokens"][b])


# ------------------------------------------------------------------ special cases


def test_orthogonal_2x2_blocks_reduce_to_average_pooling(oracle_mod):
    # a grid constant on aligned 2x2 blocks whose block vectors are mutually orthogonal:
    # reducing to a quarter of the tokens must be exactly 2x2 pooling with all sizes 4
    H = W = 8
    blocks = np.eye(16, dtype=np.float32) * np.arange(1, 17, dtype=np.float32)[:, None]
    x = np.zeros((1, H, W, 16), np.float32)
    for bh in range(4):
        for bw in range(4):
            x[0, 2 * bh:2 * bh + 2, 2 * bw:2 * bw + 2] = blocks[bh * 4 + bw]
    r = oracle_mod.oim(x, target=16)
    assert r["grid"] == (4, 4)
    assert np.all(r["sizes"] == 4)
    np.testing.assert_allclose(r["tokens"][0], blocks.astype(np.float64), atol=1e-12)
    hh, ww = np.divmod(np.arange(H * W), W)
    assert np.array_equal(r["map"][0], (hh // 2) * 4 + ww // 2)


def test_constant_grid_merges_lowest_positions_and_prefers_left(oracle_mod):
    # all cosines are 1: ties go to the lowest position, and to the left neighbour
    x = np.ones((1, 1, 7, 4), np.float32)
    r = oracle_mod.oim(x, out_hw=(1, 5))
    # positions 0 and 2 are merged, both into position 1 (0 has only a right neighbour;
    # 2 ties between 1 and 3 and takes the left one)
    assert r["trace"][0].tolist() == [0 * 2 + 1, 2 * 2 + 0]
    assert r["sizes"][0].tolist() == [3, 1, 1, 1, 1]
    assert r["map"][0].tolist() == [0, 0, 0, 1, 2, 3, 4]


def test_zero_vectors_have_zero_similarity(oracle_mod):
    x = np.zeros((1, 1, 5, 3), np.float32)
    x[0, 0, 3] = [1, 2, 3]
    x[0, 0, 4] = [1, 2, 3.5]
    r = oracle_mod.oim(x, out_hw=(1, 4))
    # only the pair (4 -> 3) has a non-zero cosine
    assert r["trace"][0].tolist() == [4 * 2 + 0]


def test_width_step_equals_height_step_on_the_transposed_grid(oracle_mod):
    x = _rand_grid(1, 6, 7, 10, seed=11)
    a = oracle_mod.oim(x, out_hw=(3, 4))
    b = oracle_mod.oim(np.ascontiguousarray(x.transpose(0, 2, 1, 3)), out_hw=(4, 3), height_first=True)
    ta = a["tokens"][0].reshape(3, 4, 10)
    tb = b["tokens"][0].reshape(4, 3, 10).transpose(1, 0, 2)
    np.testing.assert_allclose(ta, tb, rtol=0, atol=1e-13)
    ma = a["map"][0].reshape(6, 7)
    mb = b["map"][0].reshape(7, 6).T
    assert np.array_equal(ma // 4, mb % 3) and np.array_equal(ma % 4, mb // 3)


# ------------------------------------------------------------------ brute force


def _brute_force_step(grid, sizes, axis, m):
    """All ways to pick m even-position cells of every line and a neighbour for each;
    return the plan with the largest total cosine (lines are independent)."""
    h, w, D = grid.shape
    if axis == 1:
        g, s = _brute_force_step(grid.transpose(1, 0, 2), sizes.T, 0, m)
        return g.transpose(1, 0, 2), s.T
    new = np.zeros((h, w - m, D))
    news = np.zeros((h, w - m), np.int64)
    for r in range(h):
        evens = list(range(0, w, 2))
        best, best_plan = -np.inf, None
        for subset in itertools.combinations(evens, m):
            options = [[d for d in (-1, +1) if 0 <= a + d < w] for a in subset]
            for dirs in itertools.product(*options):
                tot = sum(_cos(grid[r, a], grid[r, a + d]) for a, d in zip(subset, dirs))
                if tot > best + 1e-15:
                    best, best_plan = tot, list(zip(subset, dirs))
        vec = {j: sizes[r, j] * grid[r, j] for j in range(w)}
        sz = {j: sizes[r, j] for j in range(w)}
        for a, d in best_plan:
            vec[a + d] = vec[a + d] + sizes[r, a] * grid[r, a]
            sz[a + d] += sizes[r, a]
        keep = [j for j in range(w) if j not in {a for a, _ in best_plan}]
        for o, j in enumerate(keep):
            new[r, o] = vec[j] / sz[j]
            news[r, o] = sz[j]
    return new, news


@pytest.mark.parametrize("H,W,Hf,Wf", [(4, 4, 2, 2), (3, 4, 2, 2), (4, 3, 2, 1), (2, 4, 1, 3), (4, 4, 3, 1)])
def test_plan_maximises_total_similarity_on_tiny_grids(oracle_mod, H, W, Hf, Wf):
    for seed in range(6):
        x = _rand_grid(1, H, W, 5, seed=seed)
        r = oracle_mod.oim(x, out_hw=(Hf, Wf))
        grid = x[0].astype(np.float64)
        sizes = np.ones((H, W), np.int64)
        for axis, m in oracle_mod.oim_schedule(H, W, Hf, Wf):
            grid, sizes = _brute_force_step(grid, sizes, axis, m)
        np.testing.assert_allclose(r["tokens"][0].reshape(Hf, Wf, 5), grid, rtol=1e-12, atol=1e-12)
        assert np.array_equal(r["sizes"][0].reshape(Hf, Wf), sizes)


def _anyres_golden():
    plans, scheds = [], []
    for line in open(os.path.join(GOLDEN, "oim_anyres_schedules.txt")):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "P":
            plans.append(tuple(int(v) for v in f[1:]))
        else:
            scheds.append((tuple(int(v) for v in f[1:7]), [tuple(int(v) for v in st.split(":")) for st in f[7:]]))
    return plans, scheds


def test_per_axis_merge_numbers_follow_the_hand_counted_schedules(oracle_mod):
    plans, scheds = _anyres_golden()
    assert len(plans) >= 3 and len(scheds) >= 3
    for H, W, ops, r, r_h, r_w, Hf, Wf, steps in plans:
        assert oracle_mod.oim_anyres_plan(H, W, ops, r) == ((r_h, r_w), (Hf, Wf))
        assert len(oracle_mod.oim_schedule(H, W, Hf, Wf, r=(r_h, r_w))) == steps
    for (H, W, Hf, Wf, r_h, r_w), steps in scheds:
        assert oracle_mod.oim_schedule(H, W, Hf, Wf, r=(r_h, r_w)) == steps
    with pytest.raises(ValueError):
        oracle_mod.oim_anyres_plan(8, 40, 4, 2)          # the long side would lose 4 x 10 = 40 cells, all it has


def test_per_axis_merge_numbers_keep_the_invariants(oracle_mod):
    # a 6 x 14 grid with 1 cell per column step and 3 per row step: every line loses exactly its
    # axis' number, sizes add up, merged tokens are the means of their sources
    x = _rand_grid(2, 6, 14, 7, seed=31)
    r = oracle_mod.oim(x, out_hw=(4, 8), r=(1, 3))
    assert r["sizes"].sum(axis=1).tolist() == [84, 84]
    per_line = [(0, 3), (1, 1), (0, 3), (1, 1)]
    assert oracle_mod.oim_schedule(6, 14, 4, 8, r=(1, 3)) == per_line
    assert r["trace"].shape[1] == 6 * 3 + 11 * 1 + 5 * 3 + 8 * 1
    for b in range(2):
        flat = x[b].reshape(84, 7).astype(np.float64)
        for c in range(32):
            src = np.nonzero(r["map"][b] == c)[0]
            assert len(src) == r["sizes"][b, c]
            np.testing.assert_allclose(r["tokens"][b, c], flat[src].mean(axis=0), rtol=1e-12, atol=1e-12)
    # the same merge number on both axes, given as a pair, is the plain call
    a = oracle_mod.oim(x, out_hw=(4, 8), r=(2, 2))
    b_ = oracle_mod.oim(x, out_hw=(4, 8), r=2)
    np.testing.assert_array_equal(a["map"], b_["map"])


# ------------------------------------------------------------------ replay


def test_replay_accepts_own_trace_and_flags_a_wrong_one(oracle_mod):
    x = _rand_grid(2, 6, 6, 8, seed=9)
    run = oracle_mod.oim(x, target=9)
    assert np.all(run["stats"][:, 0] > 1e-6)
    again = oracle_mod.oim(x, target=9, trace=run["trace"])
    assert np.all(again["stats"][:, 2:] == 0)
    np.testing.assert_array_equal(again["map"], run["map"])
    np.testing.assert_array_equal(again["tokens"], run["tokens"])
    # flip one direction where both neighbours exist and the margin is large: must be a violation
    bad = run["trace"].copy()
    for i, t in enumerate(bad[0][:6]):
        if 2 <= (t >> 1) <= 3:
            bad[0][i] = t ^ 1
            break
    else:
        bad[0][0] = 4 * 2  # choose another candidate outright
    flagged = oracle_mod.oim(x, target=9, trace=bad, tol=1e-9)
    assert flagged["stats"][0, 2] > 0


def _line_of_unit_vectors(angles):
    """One row of 2-D unit vectors at the given angles: the cosine of two cells is cos(angle difference)."""
    a = np.asarray(angles, dtype=np.float64)
    return np.stack([np.cos(a), np.sin(a)], axis=-1).astype(np.float32)[None, None]      # [1, 1, len, 2]


def test_replay_selection_rule_on_a_line_with_known_margins(oracle_mod):
    # Section 3.2's matching on one line of seven cells.  Even cells and their best neighbour:
    #   cell 0 -> right, cos 0.1 = 0.99500;  cell 2 -> right, cos 0.3 = 0.95534 (left: cos 0.4)
    #   cell 4 -> right, cos 0.5 = 0.87758 (left: cos 0.7);  cell 6 -> left, cos 1.0 = 0.54030
    x = _line_of_unit_vectors([0.0, 0.1, 0.5, 0.8, 1.5, 2.0, 3.0])
    own = oracle_mod.oim(x, out_hw=(1, 6))
    assert own["trace"][0].tolist() == [0 * 2 + 1]
    np.testing.assert_allclose(own["stats"][0, 0], 0.9950041652780258 - 0.955336489125606, atol=1e-6)
    # a trace that merges cell 2 instead of cell 0: the chosen score is 0.03967 below the best unchosen one
    swapped = np.array([[2 * 2 + 1]], np.int32)
    margin = 0.9950041652780258 - 0.955336489125606
    strict = oracle_mod.oim(x, out_hw=(1, 6), trace=swapped, tol=margin - 1e-3)
    assert strict["stats"][0, 2] > 0
    lenient = oracle_mod.oim(x, out_hw=(1, 6), trace=swapped, tol=margin + 1e-3)
    assert lenient["stats"][0, 2] == 0 and lenient["stats"][0, 3] > 0          # accepted, but noted as a deviation
    assert lenient["map"][0].tolist() == [0, 1, 2, 2, 3, 4, 5]                  # and the replay applied the trace's merge
    # two merges per line: {0, 4} instead of {0, 2}; the margin is cos 0.3 - cos 0.5 = 0.07775
    own2 = oracle_mod.oim(x, out_hw=(1, 5))
    assert sorted(own2["trace"][0].tolist()) == [1, 5]
    swapped2 = np.array([[0 * 2 + 1, 4 * 2 + 1]], np.int32)
    margin2 = 0.955336489125606 - 0.8775825618903728
    assert oracle_mod.oim(x, out_hw=(1, 5), trace=swapped2, tol=margin2 - 1e-3)["stats"][0, 2] > 0
    assert oracle_mod.oim(x, out_hw=(1, 5), trace=swapped2, tol=margin2 + 1e-3)["stats"][0, 2] == 0
    # the same swap along the other axis (a single column)
    xt = np.ascontiguousarray(x.transpose(0, 2, 1, 3))
    assert oracle_mod.oim(xt, out_hw=(6, 1), trace=swapped, tol=margin - 1e-3)["stats"][0, 2] > 0
    assert oracle_mod.oim(xt, out_hw=(6, 1), trace=swapped, tol=margin + 1e-3)["stats"][0, 2] == 0


def test_config0_shapes_and_near_ties(oracle_mod):
    x = gi.oim_input(0).numpy()
    r = oracle_mod.oim(x, target=144)
    assert r["grid"] == (12, 12) and r["sizes"].sum() == 576
    # smooth high-dimensional fields make near-ties common: the reason the GPU comparison
    # replays decisions instead of demanding an identical map everywhere
    assert r["stats"][0, 0] < 1e-3


def test_value_enhancement_is_the_log_of_the_size(oracle_mod):
    # Eq. 2 with uniform attention over n tokens: a token of size s with bias log s weighs like s unit tokens
    v = np.array([[[1.0, 2.0], [3.0, 5.0]]])
    s = np.array([[1, 4]])
    e = oracle_mod.oim_value_enhance(v, s)
    np.testing.assert_allclose(e[0, 0], v[0, 0])                      # log 1 = 0
    np.testing.assert_allclose(e[0, 1] - v[0, 1], np.log(4.0))
    np.testing.assert_allclose(np.exp(e - v)[0, :, 0], s[0])          # the bias exponentiates back to the size
    # hand values of Eq. 2's bias: ln 2, ln 3, ln 4 typed in
    v = np.zeros((1, 4, 1))
    e = oracle_mod.oim_value_enhance(v, np.array([[1, 2, 3, 4]]))
    np.testing.assert_allclose(e[0, :, 0], [0.0, 0.6931471805599453, 1.0986122886681098, 1.3862943611198906],
                               rtol=0, atol=1e-15)
    e = oracle_mod.oim_value_enhance(np.array([[[-0.25, 7.0]]]), np.array([[4]]))
    np.testing.assert_allclose(e[0, 0], [1.1362943611198906, 8.386294361119891], rtol=0, atol=1e-15)

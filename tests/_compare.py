"""Comparators between the CUDA path and the CPU oracle (test side only)."""
import numpy as np

DECISION_TOL = 1e-4     # cosine / relative-score margin below which a decision may differ


def value_bound(ref, dtype_name):
    """Largest accepted |got - ref|.

    fp32 I/O: 1e-5 relative + 1e-5 absolute.  bf16 I/O: the stated tolerance (2e-3 relative + 1e-3
    absolute) is about the fp32-accumulated value; storing it as bf16 adds up to half a bf16 ulp
    (2^-8 of the binade), which even a correctly rounded result cannot avoid.  The bound used here is
    tighter than that sum: half a bf16 ulp plus 1e-5 relative + 1e-6 absolute for the fp32 arithmetic."""
    a = np.abs(ref)
    if dtype_name != "bf16":
        return 1e-5 + 1e-5 * a
    half_ulp = 2.0 ** (np.floor(np.log2(np.maximum(a, 2.0 ** -126))) - 8)
    bound = half_ulp + 1e-5 * a + 1e-6
    assert np.all(bound <= 1e-3 + 2e-3 * a + half_ulp)
    return bound


def assert_values_close(got, ref, dtype_name, what):
    err = np.abs(got.astype(np.float64) - ref)
    bound = value_bound(ref, dtype_name)
    bad = err > bound
    assert not bad.any(), "%s: %d values out of tolerance, worst excess %.3g" % (
        what, int(bad.sum()), float((err - bound).max()))


def check_oim_against_oracle(oracle, x_host, gpu_tokens, gpu_sizes, gpu_map, gpu_trace, dtype_name, *,
                             target=None, out_hw=None, r=2, height_first=False, images=None,
                             matching="adjacent"):
    """x_host: float32 numpy [B,H,W,D] holding exactly the values the GPU read.
    Replays the GPU's decisions in double precision: each must be the oracle's own or tie with it
    within DECISION_TOL; the map and sizes must then equal the replayed ones exactly and the tokens
    within the value tolerance.  Images whose smallest oracle margin exceeds DECISION_TOL must
    match the oracle's free run bit for bit.  Returns the number of images that did."""
    B = x_host.shape[0]
    images = list(range(B)) if images is None else list(images)
    xs = x_host[images]
    kw = dict(target=target, out_hw=out_hw, r=r, height_first=height_first, matching=matching)
    free = oracle.oim(xs, **kw)
    replay = oracle.oim(xs, trace=gpu_trace[images], tol=DECISION_TOL, **kw)
    exact = 0
    for k, b in enumerate(images):
        assert replay["stats"][k, 2] == 0, "image %d: %d decisions outside the tolerance" % (b, replay["stats"][k, 2])
        np.testing.assert_array_equal(gpu_map[b], replay["map"][k], err_msg="image %d map" % b)
        np.testing.assert_array_equal(gpu_sizes[b], replay["sizes"][k], err_msg="image %d sizes" % b)
        assert_values_close(gpu_tokens[b], replay["tokens"][k], dtype_name, "image %d tokens" % b)
        if min(free["stats"][k, 0], free["stats"][k, 1]) > DECISION_TOL:
            np.testing.assert_array_equal(gpu_map[b], free["map"][k], err_msg="image %d map (decisive margins)" % b)
            np.testing.assert_array_equal(gpu_trace[b], free["trace"][k])
            exact += 1
    return exact


def check_oim_invariants(x_host, gpu_tokens, gpu_sizes, gpu_map, dtype_name, grid_in, grid_out, local=True):
    """Properties that hold at any size: sizes are the map's histogram and sum to H*W, every merged
    token is the mean of its sources, and (local=True: adjacent matching, where a cell only ever
    merges into a neighbour) no token moves against the compaction."""
    (H, W), (Hf, Wf) = grid_in, grid_out
    B, T = gpu_sizes.shape
    hh, ww = np.divmod(np.arange(H * W), W)
    for b in range(B):
        m = gpu_map[b]
        assert m.min() >= 0 and m.max() < T
        counts = np.bincount(m, minlength=T)
        np.testing.assert_array_equal(counts, gpu_sizes[b])
        assert counts.sum() == H * W
        sums = np.zeros((T, x_host.shape[-1]), np.float64)
        np.add.at(sums, m, x_host[b].reshape(H * W, -1).astype(np.float64))
        assert_values_close(gpu_tokens[b], sums / counts[:, None], dtype_name, "image %d means" % b)
        if local:
            hf, wf = np.divmod(m, Wf)
            assert np.all(hf <= hh) and np.all(hf >= hh - (H - Hf))
            assert np.all(wf <= ww) and np.all(wf >= ww - (W - Wf))


def check_spu_selection(scores_ref, gpu_idx, keep):
    """scores_ref: oracle energies of one sequence.  Tokens clearly above the cut must be kept,
    tokens clearly below must be dropped, the count is exact and the order ascending."""
    N = scores_ref.shape[0]
    idx = np.asarray(gpu_idx)
    assert idx.shape == (keep,)
    assert np.all(np.diff(idx) > 0) and idx.min() >= 0 and idx.max() < N
    order = np.sort(scores_ref)[::-1]
    tau_in = order[keep - 1]
    tau_out = order[keep] if keep < N else -np.inf
    kept = np.zeros(N, bool)
    kept[idx] = True
    must_keep = scores_ref > tau_out * (1 + DECISION_TOL) if keep < N else np.ones(N, bool)
    must_drop = scores_ref < tau_in * (1 - DECISION_TOL)
    assert np.all(kept[must_keep]), "%d clearly-high tokens were dropped" % int((~kept[must_keep]).sum())
    assert not np.any(kept[must_drop]), "%d clearly-low tokens were kept" % int(kept[must_drop].sum())
    return bool(keep == N or tau_in > tau_out * (1 + DECISION_TOL))   # True: the kept set is unique


def assert_scores_close(gpu_scores, ref, what="scores", median_tol=1e-5):
    """Energies of Eq. 8 against the oracle's.  A score is the norm of a filtered signal (Eq. 7) that,
    next to a strong token, is a sum of large ringing terms of both signs: arithmetic that carries
    16-17 significant bits per operand (fp32 accumulation of bf16-pair products, 2^-17 = 7.6e-6)
    is exact relative to those TERMS, not to their sum, which can be a hundred times smaller in a
    null of the ringing.  So the bound is 1e-4 of the score itself plus 1e-5 of the largest score
    within 32 tokens (circular); half of all scores must still agree to `median_tol` of themselves
    (1e-5 on the factored paths; the dense band contractions, whose N-term sums are accumulated in tensor
    memory with truncating fp32 additions, are given the full 1e-4 by the tests that reach them with long
    sequences)."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(gpu_scores, dtype=np.float64)
    n = ref.shape[0]
    local = ref.copy()
    for shift in range(1, min(32, n - 1) + 1):
        local = np.maximum(local, np.maximum(np.roll(ref, shift), np.roll(ref, -shift)))
    err = np.abs(got - ref)
    bound = 1e-4 * np.abs(ref) + 1e-5 * local
    worst = float((err / (np.abs(ref) + 1e-30)).max()) if n else 0.0
    assert np.all(err <= bound), "%s: worst relative error %.3g" % (what, worst)
    if n >= 16:
        assert np.median(err / (np.abs(ref) + 1e-30)) <= median_tol, "%s: median relative error too large" % what

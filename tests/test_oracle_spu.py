"""Pins for the SPU oracle: the DFT against a library FFT and the plain sum, Parseval,
the mask's fixed points, closed-form signals, and the order-preserving selection (CPU only)."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _signal(N, D, seed):
    return np.random.default_rng(seed).standard_normal((N, D)).astype(np.float32)


# ------------------------------------------------------------------ transform


@pytest.mark.parametrize("N", [1, 2, 3, 8, 12, 17, 36, 45, 64, 100])
def test_naive_dft_and_own_fft_match_numpy(oracle_mod, N):
    x = np.random.default_rng(N).standard_normal(N)
    ref = np.fft.fft(x)
    np.testing.assert_allclose(oracle_mod.dft_naive(x), ref, atol=1e-10)
    np.testing.assert_allclose(oracle_mod.fft(x), ref, atol=1e-10)
    z = x + 1j * np.roll(x, 1)
    np.testing.assert_allclose(oracle_mod.fft(z, inverse=True) / N, np.fft.ifft(z), atol=1e-12)


@pytest.mark.parametrize("N", [144, 1296, 2592, 4096])
def test_own_fft_on_the_workload_lengths(oracle_mod, N):
    x = np.random.default_rng(N).standard_normal(N)
    np.testing.assert_allclose(oracle_mod.fft(x), np.fft.fft(x), atol=1e-8)


@pytest.mark.parametrize("N,D,sigma", [(16, 3, 2), (45, 4, 7), (64, 5, 32), (30, 2, 0)])
def test_fft_path_equals_plain_sums(oracle_mod, N, D, sigma):
    x = _signal(N, D, 1)
    a = oracle_mod.spu_scores(x, sigma, method="naive")
    b = oracle_mod.spu_scores(x, sigma, method="fft")
    np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)
    c = oracle_mod.spu_scores_at(x, sigma, np.arange(N))
    np.testing.assert_allclose(a, c, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("N,sigma,hamming", [(48, 5, True), (49, 12, True), (48, 24, False)])
def test_scores_equal_library_filtering(oracle_mod, N, sigma, hamming):
    x = _signal(N, 6, 2)
    M = oracle_mod.spu_mask(N, sigma, hamming)
    filt = np.fft.ifft(np.fft.fft(x.astype(np.float64), axis=0) * M[:, None], axis=0)
    assert np.abs(filt.imag).max() < 1e-12          # two-sided, even mask: the output is real
    np.testing.assert_allclose(oracle_mod.spu_scores(x, sigma, hamming), np.linalg.norm(filt.real, axis=1),
                               rtol=1e-11)


def test_parseval(oracle_mod):
    N, D, sigma = 60, 7, 9
    x = _signal(N, D, 3)
    E = oracle_mod.spu_scores(x, sigma)
    M = oracle_mod.spu_mask(N, sigma)
    X = np.fft.fft(x.astype(np.float64), axis=0)
    assert np.isclose((E ** 2).sum(), (M[:, None] ** 2 * np.abs(X) ** 2).sum() / N, rtol=1e-12)


# ------------------------------------------------------------------ mask


def test_mask_fixed_points(oracle_mod):
    for N in (9, 16, 144, 1297):
        sigma = N // 2
        M = oracle_mod.spu_mask(N, sigma)
        assert M[0] == 1.0                                   # a constant signal passes unchanged
        f = np.where(np.arange(N) <= N // 2, np.arange(N), np.arange(N) - N)
        np.testing.assert_allclose(M, 0.54 + 0.46 * np.cos(2 * np.pi * f / (N - 1)), atol=1e-15)
        np.testing.assert_allclose(M[1:], M[1:][::-1], atol=1e-15)   # even in the signed frequency
        if N % 2 == 1:
            assert np.isclose(M[(N - 1) // 2], 0.08)                 # Hamming's edge value
    M = oracle_mod.spu_mask(64, 5)
    assert np.all(M[6:59] == 0) and np.all(M[:6] > 0) and np.all(M[59:] > 0)
    assert np.array_equal(oracle_mod.spu_mask(64, 5, hamming=False), (M > 0).astype(float))
    assert oracle_mod.spu_mask(1, 0).tolist() == [1.0]


def test_mask_is_the_textbook_hamming_window_centred_on_dc(oracle_mod):
    rows = [l.split() for l in open(os.path.join(GOLDEN, "hamming_window.txt")) if l[0] != "#"]
    w = np.array([float(v) for _, v in rows])
    N = len(w)
    M = oracle_mod.spu_mask(N, N // 2)
    # shifting the zero frequency to the centre of the window recovers w[n]
    np.testing.assert_allclose(np.fft.fftshift(M), w, atol=1e-14)


def test_sigma_from_cutoff(oracle_mod):
    assert oracle_mod.spu_sigma(144, 0.125) == 9
    assert oracle_mod.spu_sigma(1296, 0.125) == 81
    assert oracle_mod.spu_sigma(16384, 0.05) == 409
    assert oracle_mod.spu_sigma(16384, 0.25) == 2048
    assert oracle_mod.spu_sigma(64, None) == 4
    assert oracle_mod.spu_sigma(7, 1.0) == 3


# ------------------------------------------------------------------ closed forms


def test_constant_sequence_passes_unchanged(oracle_mod):
    N, D = 40, 5
    a = np.arange(1, D + 1, dtype=np.float32)
    x = np.tile(a, (N, 1))
    E = oracle_mod.spu_scores(x, 3)
    np.testing.assert_allclose(E, np.linalg.norm(a.astype(np.float64)), rtol=1e-12)
    assert oracle_mod.spu_select(E * 0 + 1.0, 7).tolist() == list(range(7))   # all tied: lowest indices


def test_single_cosine_in_and_out_of_band(oracle_mod):
    N, D, sigma, f0 = 64, 4, 6, 5
    a = np.array([1.0, -2.0, 0.5, 3.0])
    n = np.arange(N)
    phase = 0.3
    x = (a[None, :] * np.cos(2 * np.pi * f0 * n / N + phase)[:, None]).astype(np.float64)
    M = oracle_mod.spu_mask(N, sigma)
    E = oracle_mod.spu_scores(x, sigma)
    ref = M[f0] * np.linalg.norm(a.astype(np.float32)) * np.abs(np.cos(2 * np.pi * f0 * n / N + phase))
    np.testing.assert_allclose(E, ref, atol=2e-6)          # inputs are rounded to float32
    x_out = a[None, :] * np.cos(2 * np.pi * (sigma + 1) * n / N)[:, None]
    assert oracle_mod.spu_scores(x_out, sigma).max() < 2e-6


def test_impulse_response_and_shift(oracle_mod):
    N, D, sigma, n0 = 50, 3, 8, 17
    a = np.array([2.0, -1.0, 0.5], np.float32)
    x = np.zeros((N, D), np.float32)
    x[n0] = a
    E = oracle_mod.spu_scores(x, sigma)
    M = oracle_mod.spu_mask(N, sigma)
    n = np.arange(N)
    h = (1 + 2 * sum(M[f] * np.cos(2 * np.pi * f * (n - n0) / N) for f in range(1, sigma + 1))) / N
    np.testing.assert_allclose(E, np.linalg.norm(a) * np.abs(h), atol=1e-12)
    assert oracle_mod.spu_select(E, 1).tolist() == [n0]
    # circular shift of the input shifts the scores
    y = _signal(N, 4, 8)
    np.testing.assert_allclose(np.roll(oracle_mod.spu_scores(y, sigma), 5),
                               oracle_mod.spu_scores(np.roll(y, 5, axis=0), sigma), atol=1e-12)


def test_full_band_without_window_is_the_plain_token_norm(oracle_mod):
    for N in (31, 32):
        x = _signal(N, 9, N)
        E = oracle_mod.spu_scores(x, N // 2, hamming=False)
        np.testing.assert_allclose(E, np.linalg.norm(x.astype(np.float64), axis=1), rtol=1e-12)


# ------------------------------------------------------------------ selection


def test_select_keeps_order_and_breaks_ties_by_index(oracle_mod):
    E = np.array([3.0, 9.0, 1.0, 9.0, 5.0, 5.0, 0.5, 5.0])
    assert oracle_mod.spu_select(E, 1).tolist() == [1]
    assert oracle_mod.spu_select(E, 2).tolist() == [1, 3]
    assert oracle_mod.spu_select(E, 3).tolist() == [1, 3, 4]
    assert oracle_mod.spu_select(E, 4).tolist() == [1, 3, 4, 5]
    assert oracle_mod.spu_select(E, 8).tolist() == list(range(8))
    assert oracle_mod.spu_select(E, 0).tolist() == []
    rng = np.random.default_rng(0)
    for _ in range(20):
        E = rng.standard_normal(200) ** 2
        k = int(rng.integers(1, 200))
        idx = oracle_mod.spu_select(E, k)
        assert len(idx) == k and np.all(np.diff(idx) > 0)
        assert set(idx.tolist()) == set(np.argsort(-E, kind="stable")[:k].tolist())


def test_spu_end_to_end_gathers_original_rows(oracle_mod):
    x = _signal(2 * 36, 8, 4).reshape(2, 36, 8)
    r = oracle_mod.spu(x, cutoff=0.25, keep=9)
    assert r["sigma"] == 4
    for b in range(2):
        assert np.all(np.diff(r["idx"][b]) > 0)
        np.testing.assert_array_equal(r["hidden"][b], x[b][r["idx"][b]])   # the unfiltered tokens


def test_cascade_is_the_composition_of_single_prunes(oracle_mod):
    x = _signal(60, 6, 9)[None]
    r = oracle_mod.spu_cascade(x, (30, 12, 5), (0.5, 0.25, 1.0))
    a = oracle_mod.spu(x, cutoff=0.5, keep=30)
    b = oracle_mod.spu(a["hidden"], cutoff=0.25, keep=12)
    c = oracle_mod.spu(b["hidden"], cutoff=1.0, keep=5)
    np.testing.assert_array_equal(r["idx"][0], a["idx"][0][b["idx"][0]][c["idx"][0]])
    np.testing.assert_array_equal(r["hidden"], x[:, r["idx"][0]])
    assert np.all(np.diff(r["idx"][0]) > 0)                      # the original order survives every stage

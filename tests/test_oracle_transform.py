"""Pins for the oracle's transform, filter, score and energy functions.

Each test checks the oracle against something fixed by the paper's equations or
by mathematics, not against the oracle itself: closed forms, orthonormality,
Parseval, the gamma = 1 and omega = 0 limits, textbook statistics.
"""
import math
import os

import numpy as np
import pytest

from oracle import flashcache_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


def test_golden_dct4_ramp():
    g = _read_golden("dct4_ramp.txt")
    x = g["x"][:, None]
    for fwd, inv in ((O.dct_literal, O.idct_literal), (O.dct_fft, O.idct_fft)):
        C = fwd(x)
        np.testing.assert_allclose(C[:, 0], g["C"], atol=1e-13)
        xb = inv(O.lowpass(C, 1))
        np.testing.assert_allclose(xb[:, 0], g["x_base_omega1"], atol=1e-13)


def test_closed_forms_n1_n2():
    # N = 1: the only basis vector is the constant 1, alpha = 1.
    np.testing.assert_allclose(O.dct_literal(np.array([[3.25]])), [[3.25]], atol=0)
    # N = 2: C0 = (x0+x1)/sqrt2, C1 = (x0-x1) cos(pi/4) = (x0-x1)/sqrt2.
    x = np.array([[1.5], [-0.25]])
    C = O.dct_literal(x)
    np.testing.assert_allclose(C[:, 0], [(1.5 - 0.25) / math.sqrt(2), (1.5 + 0.25) / math.sqrt(2)], atol=1e-15)


@pytest.mark.parametrize("N", [1, 2, 3, 5, 8, 17, 64])
def test_basis_is_orthonormal(N):
    B = O.alpha(N)[:, None] * O.phi(N)
    np.testing.assert_allclose(B @ B.T, np.eye(N), atol=1e-13)
    np.testing.assert_allclose(B.T @ B, np.eye(N), atol=1e-13)


@pytest.mark.parametrize("N", [6, 16, 33])
def test_dct_of_basis_vector_is_a_delta(N):
    # sum_i phi(m0,i) phi(m,i) = N/2 delta (N for m0 = 0), so C = alpha*that.
    for m0 in (0, 1, N // 2, N - 1):
        x = O.phi(N)[m0][:, None]
        C = O.dct_literal(x)[:, 0]
        want = np.zeros(N)
        want[m0] = math.sqrt(N) if m0 == 0 else math.sqrt(N / 2.0)
        np.testing.assert_allclose(C, want, atol=1e-12)


@pytest.mark.parametrize("N", [5, 12])
def test_dct_of_unit_impulse_reads_the_basis_column(N):
    # x = delta at i0  =>  C[m] = alpha[m] cos(pi m (2 i0 + 1) / (2N)):
    # catches a swapped (m, i) or a missing half-sample shift.
    for i0 in (0, 1, N - 1):
        x = np.zeros((N, 1))
        x[i0] = 1.0
        m = np.arange(N)
        want = np.where(m == 0, math.sqrt(1 / N), math.sqrt(2 / N)) * np.cos(math.pi * m * (2 * i0 + 1) / (2 * N))
        np.testing.assert_allclose(O.dct_literal(x)[:, 0], want, atol=1e-14)
        np.testing.assert_allclose(O.dct_fft(x)[:, 0], want, atol=1e-14)


@pytest.mark.parametrize("N", [1, 2, 3, 7, 16, 31, 100, 257])
def test_literal_equals_library_tier(N):
    rng = np.random.default_rng(N)
    X = rng.standard_normal((N, 6))
    C1, C2 = O.dct_literal(X), O.dct_fft(X)
    np.testing.assert_allclose(C1, C2, atol=1e-11)
    np.testing.assert_allclose(O.idct_literal(C1), X, atol=1e-11)
    np.testing.assert_allclose(O.idct_fft(C1), X, atol=1e-11)
    for gamma in (0.0, 0.2, 0.55, 1.0):
        d1, e1 = O.score_head(X, X[::-1] * 0.5, gamma, "literal")
        d2, e2 = O.score_head(X, X[::-1] * 0.5, gamma, "fft")
        np.testing.assert_allclose(d1, d2, atol=1e-11)
        np.testing.assert_allclose(e1, e2, rtol=1e-10, atol=1e-11)


@pytest.mark.parametrize("tier", ["literal", "fft"])
def test_parseval(tier):
    rng = np.random.default_rng(1)
    X = rng.standard_normal((77, 9)) * 3.0
    C = O._TIERS[tier][0](X)
    np.testing.assert_allclose((C * C).sum(), (X * X).sum(), rtol=1e-12)
    np.testing.assert_allclose((C * C).sum(axis=0), (X * X).sum(axis=0), rtol=1e-12)


def test_cutoff_index_reading():
    assert O.cutoff_index(1024, 0.2) == 204
    assert O.cutoff_index(32768, 0.2) == 6553
    assert O.cutoff_index(10, 1.0) == 9          # clamped to N-1
    assert O.cutoff_index(10, 0.0) == 0          # DC is always kept
    assert O.cutoff_index(1, 0.2) == 0
    C = np.arange(1.0, 11.0)[:, None]
    np.testing.assert_array_equal(O.lowpass(C, 3)[:, 0], [1, 2, 3, 4, 0, 0, 0, 0, 0, 0])


@pytest.mark.parametrize("tier", ["literal", "fft"])
def test_gamma_one_reconstructs_exactly(tier):
    rng = np.random.default_rng(2)
    K, V = rng.standard_normal((40, 8)), rng.standard_normal((40, 8))
    Kb, _ = O.base_kv(K, 1.0, tier)
    np.testing.assert_allclose(Kb, K, atol=1e-12)
    dev, en = O.score_head(K, V, 1.0, tier)
    assert dev.max() < 1e-24
    assert en[0] == 0.0 and en[2] == 0.0


@pytest.mark.parametrize("tier", ["literal", "fft"])
def test_dc_only_base_is_the_column_mean(tier):
    rng = np.random.default_rng(3)
    N, d = 50, 4
    K, V = rng.standard_normal((N, d)) + 2.0, rng.standard_normal((N, d)) - 1.0
    gamma = 0.5 / N                                  # floor(gamma N) = 0
    Kb, _ = O.base_kv(K, gamma, tier)
    np.testing.assert_allclose(Kb, np.broadcast_to(K.mean(axis=0), K.shape), atol=1e-12)
    dev, en = O.score_head(K, V, gamma, tier)
    want = ((K - K.mean(0)) ** 2).mean(1) + ((V - V.mean(0)) ** 2).mean(1)
    np.testing.assert_allclose(dev, want, atol=1e-12)
    # outlier-band energy = N * population variance summed over channels
    np.testing.assert_allclose(en[0], N * K.var(axis=0).sum(), rtol=1e-12)
    np.testing.assert_allclose(en[1], (K * K).sum(), rtol=1e-12)


@pytest.mark.parametrize("tier", ["literal", "fft"])
def test_projection_is_idempotent_and_band_limited(tier):
    rng = np.random.default_rng(4)
    X = rng.standard_normal((64, 5))
    Xb, _ = O.base_kv(X, 0.25, tier)
    Xbb, Cb = O.base_kv(Xb, 0.25, tier)
    np.testing.assert_allclose(Xbb, Xb, atol=1e-12)
    assert np.abs(Cb[O.cutoff_index(64, 0.25) + 1:]).max() < 1e-12
    # scoring the Base KV against itself gives zero deviation
    dev, _ = O.score_head(Xb, Xb, 0.25, tier)
    assert dev.max() < 1e-24


def test_in_band_and_out_of_band_cosines():
    N, d, gamma = 40, 3, 0.2                        # omega = 8
    omega = O.cutoff_index(N, gamma)
    assert omega == 8
    inside = np.repeat(O.phi(N)[omega][:, None], d, axis=1)        # m = omega is kept (inclusive band)
    outside = np.repeat(O.phi(N)[omega + 1][:, None], d, axis=1)   # m = omega+1 is removed
    zero = np.zeros((N, d))
    dev_in, _ = O.score_head(inside, zero, gamma)
    dev_out, en = O.score_head(outside, zero, gamma)
    assert dev_in.max() < 1e-24
    np.testing.assert_allclose(dev_out, (outside ** 2).mean(axis=1), atol=1e-13)
    np.testing.assert_allclose(en[0], en[1], rtol=1e-12)           # all energy is outlier energy


@pytest.mark.parametrize("tier", ["literal", "fft"])
def test_score_energy_identity(tier):
    # Parseval on the removed band: d * sum_x Dev_k[x] = sum_{m > omega} P_k[m].
    rng = np.random.default_rng(5)
    N, d = 96, 16
    K, V = rng.standard_normal((N, d)), 2.0 * rng.standard_normal((N, d))
    zero = np.zeros((N, d))
    dk, ek = O.score_head(K, zero, 0.3, tier)
    dv, ev = O.score_head(zero, V, 0.3, tier)
    dboth, eboth = O.score_head(K, V, 0.3, tier)
    np.testing.assert_allclose(d * dk.sum(), ek[0], rtol=1e-12)
    np.testing.assert_allclose(d * dv.sum(), ev[2], rtol=1e-12)
    np.testing.assert_allclose(dboth, dk + dv, atol=1e-13)         # Dev = Dev_k + Dev_v, unweighted
    np.testing.assert_allclose(eboth, (ek[0], ek[1], ev[2], ev[3]), rtol=1e-12)


def test_white_noise_expectation():
    # For white noise of variance s^2 an orthogonal projection that removes r of
    # N directions leaves E[Dev_k] = s^2 (1 - r/N).
    rng = np.random.default_rng(6)
    N, d, s, gamma = 2048, 64, 0.7, 0.2
    K = s * rng.standard_normal((N, d))
    dev, _ = O.score_head(K, np.zeros((N, d)), gamma, "fft")
    r = O.cutoff_index(N, gamma) + 1
    assert abs(dev.mean() / (s * s * (1 - r / N)) - 1.0) < 0.02


def test_score_layer_packs_sequences_independently():
    rng = np.random.default_rng(7)
    lens = [13, 0, 32, 7]
    cu = np.concatenate([[0], np.cumsum(lens)])
    H, d = 3, 4
    K, V = rng.standard_normal((cu[-1], H, d)), rng.standard_normal((cu[-1], H, d))
    scores, energy = O.score_layer(K, V, cu, 0.2, "literal")
    assert scores.shape == (H, cu[-1]) and energy.shape == (4, 4)
    for b, n in enumerate(lens):
        if n == 0:
            assert not energy[b].any()
            continue
        tot = np.zeros(4)
        for h in range(H):
            dev, en = O.score_head(K[cu[b]:cu[b + 1], h], V[cu[b]:cu[b + 1], h], 0.2)
            np.testing.assert_allclose(scores[h, cu[b]:cu[b + 1]], dev, atol=1e-13)
            tot += en
        np.testing.assert_allclose(energy[b], tot, rtol=1e-12)


def test_energy_ratio():
    assert O.energy_ratio((1.0, 4.0, 3.0, 6.0)) == 0.25 + 0.5
    assert O.energy_ratio((0.0, 0.0, 3.0, 6.0)) == 0.5          # empty matrix contributes 0
    assert O.energy_ratio((0.0, 0.0, 0.0, 0.0)) == 0.0


def test_generator_structure_low_frequency_dominates():
    from paper_2511_16786_b200 import synth_kv as S
    cfg = S.paper_configs()["cfg1"]
    K, V = S.make_layer(cfg, 0)
    K2, _ = S.make_layer(cfg, 0)
    assert (K == K2).all()                                       # seeded: same bytes every time
    assert K.shape == (1024, 4, 128) and str(K.dtype) == "torch.float32"
    dev, en = O.score_head(K[:, 0].numpy(), V[:, 0].numpy(), cfg.gamma, "fft")
    assert en[0] / en[1] < 0.2                                   # most energy sits in the kept band
    # rows replaced by N(0, 5) outliers stand far above the noise floor
    top = O.select_topk(dev, 20)
    assert dev[top].min() > 20 * np.median(dev)


# ---------------------------------------------------------------- power spectrum (Eq. 11)
def test_power_spectrum_of_a_single_basis_vector_is_one_line():
    # x = a * alpha[m0] * phi_N(m0, .) in one channel has C = a * delta[m - m0] (orthonormal rows, Eq. 7),
    # so P is a^2 at m0 and zero elsewhere
    N, H, d = 37, 2, 3
    for m0 in (0, 1, 9, 36):
        K = np.zeros((N, H, d))
        V = np.zeros((N, H, d))
        m1 = (m0 + 5) % N
        K[:, 1, 2] = 3.0 * O.alpha(N)[m0] * O.phi(N)[m0]
        V[:, 0, 0] = -2.0 * O.alpha(N)[m1] * O.phi(N)[m1]
        P = O.power_spectrum(K, V, [0, N])
        want = np.zeros((N, 2))
        want[m0, 0] = 9.0
        want[m1, 1] = 4.0
        np.testing.assert_allclose(P, want, atol=1e-12)


@pytest.mark.parametrize("tier", ["literal", "fft"])
def test_power_spectrum_parseval_and_band_sums(tier):
    rng = np.random.default_rng(11)
    lens = [24, 0, 9, 16]
    cu = [0] + [int(x) for x in np.cumsum(lens)]
    K = rng.standard_normal((cu[-1], 2, 4))
    V = rng.standard_normal((cu[-1], 2, 4)) * 2.0
    P = O.power_spectrum(K, V, cu, tier)
    _, energy = O.score_layer(K, V, cu, 0.25, "literal")
    for b, n in enumerate(lens):
        if n == 0:
            continue
        s, e = cu[b], cu[b + 1]
        assert np.isclose(P[s:e, 0].sum(), (K[s:e] ** 2).sum(), rtol=1e-12)          # Parseval: orthonormal transform
        assert np.isclose(P[s:e, 1].sum(), (V[s:e] ** 2).sum(), rtol=1e-12)
        om = O.cutoff_index(n, 0.25)
        np.testing.assert_allclose([P[s + om + 1:e, 0].sum(), P[s:e, 0].sum(), P[s + om + 1:e, 1].sum(), P[s:e, 1].sum()],
                                   energy[b], rtol=1e-10)                            # the sums Eq. 12 is made of


def test_power_spectrum_tiers_agree():
    rng = np.random.default_rng(12)
    for n in (1, 2, 7, 31, 64):
        K = rng.standard_normal((n, 1, 5))
        V = rng.standard_normal((n, 1, 5))
        np.testing.assert_allclose(O.power_spectrum(K, V, [0, n], "fft"), O.power_spectrum(K, V, [0, n], "literal"),
                                   rtol=1e-9, atol=1e-12)


# ---------------------------------------------------------------- cutoff from the spectrum (Eq. 11-12)
def test_cutoff_from_spectrum_single_basis_vector_steps_at_its_frequency():
    # all the energy sits in bin m0: every share in (0, 1] gives omega = m0, and min(N-1, floor(gamma*N)) gives it back
    N, d, m0 = 96, 3, 17
    X = np.outer(O.phi(N)[m0], np.array([1.0, -2.0, 0.5]))
    P = O.power_spectrum(X.reshape(N, 1, d), np.zeros((N, 1, d)), [0, N], "literal")
    for share in (1e-6, 0.3, 0.999):
        omega, gamma = O.cutoff_for_energy_share(P, share)
        assert omega == m0
        assert O.cutoff_index(N, gamma) == omega


def test_cutoff_from_spectrum_white_noise_tracks_the_share():
    # flat expected spectrum: the kept band must hold the share, so omega + 1 is close to share * N
    rng = np.random.default_rng(5)
    N, d = 2048, 64
    K, V = rng.standard_normal((N, 1, d)), rng.standard_normal((N, 1, d))
    P = O.power_spectrum(K, V, [0, N], "fft")
    for share in (0.1, 0.5, 0.9):
        omega, _ = O.cutoff_for_energy_share(P, share)
        assert abs((omega + 1) / N - share) < 0.02


def test_cutoff_from_spectrum_is_the_eq12_threshold_and_monotone():
    # by its definition: outlier-energy share (Eq. 12 over K and V together) <= 1 - share at omega and > 1 - share at omega - 1
    rng = np.random.default_rng(6)
    N = 301
    P = rng.random((N, 2)) * np.exp(-np.arange(N) / 40.0)[:, None]
    tot = P.sum()
    prev = -1
    for share in (0.0, 0.2, 0.5, 0.8, 0.95, 1.0):
        omega, gamma = O.cutoff_for_energy_share(P, share)
        assert omega >= prev
        prev = omega
        assert P[omega + 1:].sum() / tot <= 1.0 - share + 1e-12
        if omega > 0:
            assert P[omega:].sum() / tot > 1.0 - share - 1e-12
        assert O.cutoff_index(N, gamma) == omega
    assert O.cutoff_for_energy_share(np.zeros((8, 2)), 0.5)[0] == 0
    # brute force on a tiny spectrum
    P = np.array([[1.0, 0.0], [0.0, 1.0], [2.0, 0.0], [0.0, 0.0]])
    assert [O.cutoff_for_energy_share(P, s)[0] for s in (0.25, 0.26, 0.5, 0.51, 1.0)] == [0, 1, 1, 2, 2]

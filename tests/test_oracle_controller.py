"""Pins for the oracle's gamma controller (paper Sec. 4.3, Eq. 1): hand-computed networks
with small integer weights, structural special cases and a numpy matmul cross-check."""
import numpy as np
import pytest

import oracle


def _mlp(W1, b1, W2, b2, **kw):
    return oracle.Mlp(np.array(W1, np.float32), np.array(b1, np.float32),
                      np.array(W2, np.float32), np.array(b2, np.float32), **kw)


def test_hand_computed_network_layout0():
    # features: Hbar=2, cbar=0.5, Hmax=9 (unused in layout 0), cmin=0.25, flags (1,0)
    # x = [2, 0.5, 0.25, 1, 0]
    feat = np.array([[2.0, 0.5, 9.0, 0.25]])
    comp = np.array([[1.0, 0.0]], np.float32)
    W1 = np.zeros((16, 5)); b1 = np.zeros(16)
    W1[0] = [1, 2, 4, 0, 0]; b1[0] = -1      # 2 + 1 + 1 - 1 = 3
    W1[1] = [-1, 0, 0, 1, 5]; b1[1] = 0      # -2 + 1 = -1 -> ReLU 0
    W1[2] = [0, 0, 8, -1, 0]; b1[2] = 0.5    # 2 - 1 + .5 = 1.5
    W1[15] = [0, 4, 0, 0, 0]; b1[15] = 0     # 2
    W2 = np.zeros((4, 16)); b2 = np.array([0.0, 0.5, -1.0, 0.25])
    W2[0, 0] = 1                              # o0 = 3
    W2[1, 1] = 7; W2[1, 2] = 1                # o1 = 0 + 1.5 + .5 = 2
    W2[2, 15] = 1; W2[2, 0] = 0.5             # o2 = 2 + 1.5 - 1 = 2.5
    W2[3, 2] = -2                             # o3 = -3 + .25 = -2.75
    r = oracle.select_gamma(feat, comp, _mlp(W1, b1, W2, b2))
    # Eq. 1: E = o * gamma + 1 with gamma in {2,4,6,8}
    np.testing.assert_allclose(r["scores"][0], [3 * 2 + 1, 2 * 4 + 1, 2.5 * 6 + 1, -2.75 * 8 + 1], rtol=1e-15)
    assert r["gamma_next"][0] == 6
    # raw-score mode returns the heads themselves; best head is o0
    r = oracle.select_gamma(feat, comp, _mlp(W1, b1, W2, b2, score_transform=1))
    np.testing.assert_allclose(r["scores"][0], [3, 2, 2.5, -2.75], rtol=1e-15)
    assert r["gamma_next"][0] == 2


def test_paper_context_vector_layout1_uses_hmax():
    # x = [Hbar, cbar, Hmax, cmin, comp] (Sec. 4.3); a unit that reads only Hmax
    feat = np.array([[2.0, 0.5, 9.0, 0.25]])
    comp = np.array([[2.0]], np.float32)
    W1 = np.zeros((16, 5)); b1 = np.zeros(16)
    W1[3, 2] = 1.0        # h3 = Hmax = 9
    W1[4, 4] = 3.0        # h4 = 3*comp = 6
    W2 = np.zeros((4, 16)); b2 = np.zeros(4)
    W2[0, 3] = 1; W2[3, 4] = 0.5
    r = oracle.select_gamma(feat, comp, _mlp(W1, b1, W2, b2, feature_layout=1))
    np.testing.assert_allclose(r["scores"][0], [9 * 2 + 1, 1, 1, 3 * 8 + 1], rtol=1e-15)
    assert r["gamma_next"][0] == 8


def test_zero_first_layer_reduces_to_bias_path():
    rng = np.random.default_rng(0)
    b1 = rng.integers(-3, 4, 16).astype(np.float64)
    W2 = rng.integers(-2, 3, (4, 16)).astype(np.float64)
    b2 = rng.integers(-2, 3, 4).astype(np.float64)
    feat = rng.normal(size=(7, 4)); comp = rng.integers(0, 2, (7, 2)).astype(np.float32)
    r = oracle.select_gamma(feat, comp, _mlp(np.zeros((16, 5)), b1, W2, b2, score_transform=1))
    expect = W2 @ np.maximum(b1, 0) + b2
    for b in range(7):
        np.testing.assert_allclose(r["scores"][b], expect, rtol=1e-15)


def test_ties_pick_the_smallest_gamma_and_are_flagged():
    feat = np.zeros((1, 4)); comp = np.zeros((1, 2), np.float32)
    W1 = np.zeros((16, 5)); b1 = np.zeros(16); W2 = np.zeros((4, 16))
    # all heads zero => every E = 1 => lowest index (gamma = 2)
    r = oracle.select_gamma(feat, comp, _mlp(W1, b1, W2, np.zeros(4)))
    assert r["gamma_next"][0] == 2 and r["near"][0] & oracle.NEAR_GAMMA
    # E = [1+2*.6, 1+4*.3, ...] = [2.2, 2.2, 1, 1]: exact tie in o*gamma up to rounding; use exact ones
    r = oracle.select_gamma(feat, comp, _mlp(W1, b1, W2, [0.5, 0.25, 0.0, 0.125]))
    np.testing.assert_allclose(r["scores"][0], [2, 2, 1, 2])
    assert r["gamma_next"][0] == 2
    # a clear winner is not flagged
    r = oracle.select_gamma(feat, comp, _mlp(W1, b1, W2, [0.5, 0.25, 1.0, 0.125]))
    assert r["gamma_next"][0] == 6 and not (r["near"][0] & oracle.NEAR_GAMMA)


@pytest.mark.parametrize("layout,n_comp", [(0, 2), (1, 1)])
def test_random_network_matches_numpy_matmul(layout, n_comp):
    rng = np.random.default_rng(5)
    W1 = rng.normal(0, 0.1, (16, 5)).astype(np.float32); b1 = rng.normal(0, 0.1, 16).astype(np.float32)
    W2 = rng.normal(0, 0.1, (4, 16)).astype(np.float32); b2 = rng.normal(0, 0.1, 4).astype(np.float32)
    feat = np.abs(rng.normal(size=(50, 4))); comp = rng.integers(0, 2, (50, n_comp)).astype(np.float32)
    r = oracle.select_gamma(feat, comp, oracle.Mlp(W1, b1, W2, b2, feature_layout=layout))
    if layout == 0:
        x = np.concatenate([feat[:, [0, 1, 3]], comp.astype(np.float64)], axis=1)
    else:
        x = np.concatenate([feat, comp.astype(np.float64)], axis=1)
    h = np.maximum(x @ W1.astype(np.float64).T + b1, 0)
    o = h @ W2.astype(np.float64).T + b2
    E = o * np.array([2, 4, 6, 8]) + 1
    np.testing.assert_allclose(r["scores"], E, rtol=1e-12)
    np.testing.assert_array_equal(r["gamma_next"], np.array([2, 4, 6, 8])[E.argmax(1)])


# ---- the paper's own predictor form (Sec. 4.3): f(x, gamma) -> a_hat, evaluated per candidate ----
def test_paper_form_linear_predictor_closed_form():
    # a_hat(gamma) = 0.5 - 0.06 gamma  =>  E(gamma) = gamma (0.5 - 0.06 gamma) + 1, maximal near 0.5 / 0.12 = 4.17
    feat = np.array([[1.0, 0.5, 2.0, 0.25]])
    comp = np.array([[1.0]], np.float32)
    W2 = np.array([[0.1, 0.2, 0.0, 0.4, -0.1, -0.06]], np.float32)       # [Hbar, cbar, Hmax, cmin, comp, gamma]
    m = oracle.Mlp(np.zeros((0, 6), np.float32), np.zeros(0, np.float32), W2, np.array([0.3], np.float32),
                   feature_layout=2)
    out = oracle.select_gamma(feat, comp, m)
    want = [g * (0.5 - 0.06 * g) + 1.0 for g in (2, 4, 6, 8)]
    np.testing.assert_allclose(out["scores"][0], want, rtol=1e-6)
    assert out["gamma_next"][0] == 4
    raw = oracle.select_gamma(feat, comp, oracle.Mlp(m.W1, m.b1, m.W2, m.b2, feature_layout=2, score_transform=1))
    # (weights are float32: the cancellation at gamma = 8 leaves an absolute 1e-8, not a relative 1e-6)
    np.testing.assert_allclose(raw["scores"][0], [0.5 - 0.06 * g for g in (2, 4, 6, 8)], rtol=1e-6, atol=1e-7)


def test_paper_form_hidden_units_by_hand():
    # h1 = relu(Hbar + gamma - 5), h2 = relu(7 - gamma); a_hat = 0.1 h1 + 0.05 h2; Hbar = 1
    feat = np.array([[1.0, 0.0, 0.0, 0.0]])
    W1 = np.array([[1, 0, 0, 0, 0, 1], [0, 0, 0, 0, 0, -1]], np.float32)
    b1 = np.array([-5, 7], np.float32)
    W2 = np.array([[0.1, 0.05]], np.float32)
    m = oracle.Mlp(W1, b1, W2, np.array([0.0], np.float32), feature_layout=2)
    out = oracle.select_gamma(feat, np.zeros((1, 1), np.float32), m)
    a_hat = np.array([0.25, 0.15, 0.25, 0.4])
    np.testing.assert_allclose(out["scores"][0], a_hat * np.array([2, 4, 6, 8]) + 1.0, rtol=1e-6)
    assert out["gamma_next"][0] == 8


def test_paper_form_without_gamma_dependence_picks_an_end_of_the_range():
    rng = np.random.default_rng(3)
    feat = np.abs(rng.normal(size=(50, 4)))
    comp = rng.integers(0, 3, (50, 1)).astype(np.float32)
    W1 = rng.normal(0, 0.3, (16, 6)).astype(np.float32)
    W1[:, 5] = 0                                                          # the prediction ignores gamma
    m = oracle.Mlp(W1, rng.normal(0, 0.3, 16).astype(np.float32), rng.normal(0, 0.3, (1, 16)).astype(np.float32),
                   np.array([0.01], np.float32), feature_layout=2)
    out = oracle.select_gamma(feat, comp, m)
    a_hat = (out["scores"][:, 0] - 1.0) / 2.0
    assert np.all(out["gamma_next"][a_hat > 1e-6] == 8) and np.all(out["gamma_next"][a_hat < -1e-6] == 2)
    np.testing.assert_allclose(out["scores"], a_hat[:, None] * np.array([2, 4, 6, 8]) + 1.0, rtol=1e-9, atol=1e-12)

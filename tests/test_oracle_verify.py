"""Pins for the oracle's verification: the greedy rule of paper Sec. 3.1, and the lossless
speculative-sampling rule (accept while u < min(1, p/q); residual norm(max(0, p-q)); bonus
from p) that the paper cites in Sec. 1 and 2.1.  Closed forms, brute force on tiny
vocabularies and the statistical properties the rule is known for."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle

NEG = -np.inf


def _softmax(x, T=1.0):
    return scipy.special.softmax(np.asarray(x, np.float64) / float(np.float32(T)), axis=-1)


def _broadcast_rows(a, B):
    """[P, V] logits seen as [B, P, V] with row stride 0 (every trial reads the same logits)."""
    return np.broadcast_to(a[None], (B,) + a.shape)


def test_identical_distributions_accept_everything():
    rng = np.random.default_rng(0)
    B, G, V = 64, 5, 300
    t = rng.normal(0, 2, (B, G + 1, V)).astype(np.float32)
    d = t[:, :G].copy()
    tok = rng.integers(0, V, (B, G)).astype(np.int32)
    u = rng.random((B, G + 1, 2)).astype(np.float32)
    u[0] = np.float32(1.0) - np.float32(2 ** -24)  # the largest float32 below 1
    u[1] = 0.0
    r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, uniforms=u, temperature_scalar=0.7))
    assert np.all(r["n_accepted"] == G)
    np.testing.assert_array_equal(r["out_tokens"][:, :G], tok)
    assert np.all((r["out_tokens"][:, G] >= 0) & (r["out_tokens"][:, G] < V))


def test_one_hot_draft_accepts_with_probability_alpha():
    # q is one-hot on token 0, p = (alpha', 1 - alpha'): accept iff u < alpha'
    alpha_logits = np.array([math.log(0.3), math.log(0.7)], np.float32)
    alpha = _softmax(alpha_logits)[0]
    us = np.array([0.0, 0.1, alpha - 1e-4, alpha + 1e-4, 0.9], np.float64)
    B = len(us)
    t = _broadcast_rows(np.stack([alpha_logits, alpha_logits]), B)
    d = _broadcast_rows(np.array([[5.0, NEG]], np.float32), B)
    u = np.zeros((B, 2, 2), np.float32)
    u[:, 0, 0] = us
    u[:, :, 1] = 0.5
    r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=np.zeros((B, 1), np.int32), uniforms=u))
    np.testing.assert_array_equal(r["n_accepted"], [1, 1, 1, 0, 0])
    # rejected rows resample from max(0, p - q) = (0, 1 - alpha): always token 1
    np.testing.assert_array_equal(r["out_tokens"][3:, 0], [1, 1])
    # accepted rows emit the draft token then a bonus from p at u' = 0.5 -> token 1 (alpha < .5)
    np.testing.assert_array_equal(r["out_tokens"][:3], [[0, 1]] * 3)


def test_zero_draft_probability_token_is_accepted_iff_target_allows_it():
    # q(x) = 0: u*q < p holds iff p(x) > 0 (such a token cannot be drawn from q, but callers may pass it)
    d = np.array([[[0.0, NEG, 0.0]]], np.float32)
    t = np.array([[[0.0, 0.0, 0.0], [0.0, 0.0, 0.0]]], np.float32)
    u = np.full((1, 2, 2), 0.99, np.float32)
    r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=np.array([[1]], np.int32), uniforms=u))
    assert r["n_accepted"][0] == 1
    t2 = t.copy(); t2[0, 0, 1] = NEG
    r = oracle.verify(oracle.Batch(draft=d, target=t2, draft_tokens=np.array([[1]], np.int32), uniforms=u))
    assert r["n_accepted"][0] == 0
    # residual = max(0, p - q) with p = (.5, 0, .5), q = (.5, 0, .5) -> empty; falls back to p
    assert r["out_tokens"][0, 0] in (0, 2)


def test_inverse_cdf_convention():
    w = np.array([0.0, 0.2, 0.0, 0.3, 0.5, 0.0])
    # smallest v with cumulative weight > u * W
    assert oracle.inverse_cdf(w, 0.0)[0] == 1
    assert oracle.inverse_cdf(w, 0.19)[0] == 1
    assert oracle.inverse_cdf(w, 0.21)[0] == 3
    assert oracle.inverse_cdf(w, 0.49)[0] == 3
    assert oracle.inverse_cdf(w, 0.51)[0] == 4
    assert oracle.inverse_cdf(w, 0.999999)[0] == 4
    # scale invariance and the boundary flag
    assert oracle.inverse_cdf(w * 7.0, 0.21) == (3, 0)
    assert oracle.inverse_cdf(w, 0.2 + 1e-8)[1] == 1
    assert oracle.inverse_cdf(w, 0.35)[1] == 0
    assert oracle.inverse_cdf(np.zeros(4), 0.3)[0] == -1


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_residual_sampling_histogram_on_u_grid(seed):
    # V <= 8, one drafted position that is always rejected; sweep u' over a fine grid and compare
    # the histogram of the resampled token with max(0, p - q) / R.
    rng = np.random.default_rng(seed)
    V = 8 - seed
    tl = rng.normal(0, 1.5, (2, V)).astype(np.float32)
    dl = rng.normal(0, 1.5, (1, V)).astype(np.float32)
    p, q = _softmax(tl[0]), _softmax(dl[0])
    x = int(np.argmin(p / q))          # the token with the smallest ratio
    assert p[x] < q[x]
    N = 100000
    u = np.zeros((N, 2, 2), np.float32)
    u[:, 0, 0] = np.float32(1.0) - np.float32(2 ** -24)  # rejects: ratio < 1 - 2^-24
    u[:, 0, 1] = (np.arange(N) + 0.5) / N
    r = oracle.verify(oracle.Batch(draft=_broadcast_rows(dl, N), target=_broadcast_rows(tl, N),
                                   draft_tokens=np.full((N, 1), x, np.int32), uniforms=u, n_threads=4))
    assert np.all(r["n_accepted"] == 0)
    hist = np.bincount(r["out_tokens"][:, 0], minlength=V) / N
    resid = np.maximum(0.0, p - q)
    resid /= resid.sum()
    np.testing.assert_allclose(hist, resid, atol=1e-4)
    assert np.all(hist[p <= q] == 0)


@pytest.mark.parametrize("gamma", [1, 2, 3, 4])
def test_emitted_tokens_follow_the_target_distribution(gamma):
    # V = 8, 10^6 trials.  Draft tokens are drawn from q by numpy; the token emitted at position
    # i, given that positions < i were accepted, must be distributed as p_i (lossless property).
    rng = np.random.default_rng(100 + gamma)
    V, N, T = 8, 1_000_000, 0.9
    tl = rng.normal(0, 1.2, (gamma + 1, V)).astype(np.float32)
    dl = (tl[:gamma] + rng.normal(0, 0.8, (gamma, V))).astype(np.float32)
    p, q = _softmax(tl, T), _softmax(dl, T)
    tok = np.stack([rng.choice(V, size=N, p=q[i]) for i in range(gamma)], axis=1).astype(np.int32)
    u = rng.random((N, gamma + 1, 2)).astype(np.float32)
    r = oracle.verify(oracle.Batch(draft=_broadcast_rows(dl, N), target=_broadcast_rows(tl, N),
                                   draft_tokens=tok, uniforms=u, temperature_scalar=T, n_threads=8))
    n, out = r["n_accepted"], r["out_tokens"]
    assert n.min() >= 0 and n.max() <= gamma
    for i in range(gamma + 1):
        reached = n >= i
        cnt = np.bincount(out[reached, i], minlength=V)
        chi = scipy.stats.chisquare(cnt, p[i] * reached.sum())
        assert chi.pvalue > 1e-4, (i, chi)
    # structure: accepted prefix is the draft, -1 after the fresh token
    cols = np.arange(gamma + 1)[None, :]
    np.testing.assert_array_equal(out[:, :gamma][cols[:, :gamma] < n[:, None]],
                                  tok[cols[:, :gamma] < n[:, None]])
    assert np.all(out[cols > n[:, None]] == -1)
    # the acceptance probability at position 0 is sum_v min(p, q)
    acc0 = np.minimum(p[0], q[0]).sum()
    assert (n >= 1).mean() == pytest.approx(acc0, abs=4 * math.sqrt(acc0 * (1 - acc0) / N))


@pytest.mark.parametrize("alpha_nominal,gamma", [(0.7, 4), (0.5, 8), (0.9, 6)])
def test_expected_tokens_per_step_under_iid_acceptance(alpha_nominal, gamma):
    # q one-hot on token 0 and p(0) = alpha at every position => acceptances are iid Bernoulli(alpha)
    # and E[k + 1] = (1 - alpha^(gamma+1)) / (1 - alpha)   (k + 1 tokens per step, Sec. 3.1)
    rng = np.random.default_rng(7)
    N = 1_000_000
    tl = np.tile(np.array([math.log(alpha_nominal), math.log(1 - alpha_nominal)], np.float32), (gamma + 1, 1))
    alpha = _softmax(tl[0])[0]
    dl = np.tile(np.array([0.0, NEG], np.float32), (gamma, 1))
    u = rng.random((N, gamma + 1, 2)).astype(np.float32)
    r = oracle.verify(oracle.Batch(draft=_broadcast_rows(dl, N), target=_broadcast_rows(tl, N),
                                   draft_tokens=np.zeros((N, gamma), np.int32), uniforms=u, n_threads=8))
    emitted = r["n_accepted"].astype(np.float64) + 1
    expect = (1 - alpha ** (gamma + 1)) / (1 - alpha)
    assert emitted.mean() == pytest.approx(expect, abs=4 * emitted.std() / math.sqrt(N))


def test_greedy_rule_matches_brute_force():
    rng = np.random.default_rng(11)
    B, G, V = 200, 6, 50
    t = rng.normal(0, 1, (B, G + 1, V)).astype(np.float32)
    d = rng.normal(0, 1, (B, G, V)).astype(np.float32)
    am = t.argmax(-1)
    tok = am[:, :G].astype(np.int32).copy()
    # break the match at a random position for most rows
    brk = rng.integers(0, G + 2, B)
    for b in range(B):
        if brk[b] < G:
            tok[b, brk[b]] = (tok[b, brk[b]] + 1 + rng.integers(0, V - 1)) % V
    r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok,
                                   uniforms=np.zeros((B, G + 1, 2), np.float32), temperature_scalar=0.0))
    for b in range(B):
        n = min(brk[b], G)
        assert r["n_accepted"][b] == n
        assert list(r["out_tokens"][b, :n]) == list(tok[b, :n])
        assert r["out_tokens"][b, n] == am[b, n]
        assert np.all(r["out_tokens"][b, n + 1:] == -1)


def test_greedy_ties_resolve_to_lowest_index():
    t = np.zeros((1, 2, 6), np.float32)
    t[0, 0, [2, 4]] = 3.0
    t[0, 1, [5, 1]] = 1.0
    d = np.zeros((1, 1, 6), np.float32)
    mk = lambda x: oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=np.array([[x]], np.int32),
                                              uniforms=np.zeros((1, 2, 2), np.float32), temperature_scalar=0.0))
    r = mk(2)
    assert r["n_accepted"][0] == 1 and list(r["out_tokens"][0]) == [2, 1]
    r = mk(4)
    assert r["n_accepted"][0] == 0 and list(r["out_tokens"][0]) == [2, -1]
    assert oracle.argmax_row(np.array([1, 7, 7, 7], np.float32)) == 1


def test_low_temperature_sampling_approaches_greedy():
    # tie-free rows with argmax draft tokens: as T -> 0+ the stochastic rule accepts exactly
    # where the target argmax equals the draft token and replaces with the target argmax
    rng = np.random.default_rng(12)
    B, G, V = 40, 4, 30
    # every row is a permutation of 0..V-1 (gaps >= 1), the draft a second permutation mixed in
    t = rng.permuted(np.tile(np.arange(V, dtype=np.float64), (B, G + 1, 1)), axis=-1).astype(np.float32)
    d = (t[:, :G] + 3 * rng.permuted(np.tile(np.arange(V, dtype=np.float64), (B, G, 1)), axis=-1) / V).astype(np.float32)
    tok = d.argmax(-1).astype(np.int32)
    u = (rng.random((B, G + 1, 2)) * 0.98 + 0.01).astype(np.float32)
    cold = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, uniforms=u, temperature_scalar=1e-3))
    greedy = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, uniforms=u, temperature_scalar=0.0))
    np.testing.assert_array_equal(cold["n_accepted"], greedy["n_accepted"])
    np.testing.assert_array_equal(cold["out_tokens"], greedy["out_tokens"])


def test_ragged_gamma_and_mixed_temperature_rows():
    rng = np.random.default_rng(13)
    B, G, V = 6, 8, 40
    t = rng.normal(0, 1, (B, G + 1, V)).astype(np.float32)
    d = t[:, :G].copy()                       # identical => stochastic rows accept all gamma_b
    tok = d.argmax(-1).astype(np.int32)       # and greedy rows match the target argmax
    gam = np.array([1, 2, 8, 5, 3, 8], np.int32)
    T = np.array([1.0, 0.0, 0.5, 0.0, 2.0, 1.0], np.float32)
    t[:, :, :] = np.where(np.arange(G + 1)[None, :, None] > gam[:, None, None], np.nan, t)  # unused => garbage
    d[:, :, :] = np.where(np.arange(G)[None, :, None] >= gam[:, None, None], np.nan, d)
    u = rng.random((B, G + 1, 2)).astype(np.float32)
    r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, gamma=gam, temperature=T, uniforms=u))
    assert list(r["row_status"]) == [0] * B
    np.testing.assert_array_equal(r["n_accepted"], gam)
    for b in range(B):
        assert np.all(r["out_tokens"][b, gam[b] + 1:] == -1)
        if T[b] == 0:
            assert r["out_tokens"][b, gam[b]] == np.nanargmax(t[b, gam[b]])


def test_row_status_flags_and_outputs():
    rng = np.random.default_rng(14)
    B, G, V = 6, 3, 20
    t = rng.normal(0, 1, (B, G + 1, V)).astype(np.float32)
    d = rng.normal(0, 1, (B, G, V)).astype(np.float32)
    tok = rng.integers(0, V, (B, G)).astype(np.int32)
    tok[1, 2] = V
    tok[2, 0] = -1
    t[3, 0, 4] = np.nan                     # position 0 is read whatever happens later
    gam = np.array([3, 3, 3, 3, 4, 2], np.int32)
    T = np.array([1, 1, 0, 1, 1, -0.5], np.float32)
    u = rng.random((B, G + 1, 2)).astype(np.float32)
    r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, gamma=gam, temperature=T, uniforms=u))
    assert list(r["row_status"]) == [0, oracle.ROW_BAD_TOKEN, oracle.ROW_BAD_TOKEN, oracle.ROW_NONFINITE,
                                     oracle.ROW_BAD_GAMMA, oracle.ROW_BAD_TEMPERATURE]
    assert np.all(r["n_accepted"][1:] == 0) and np.all(r["out_tokens"][1:] == -1)


def test_near_accept_flag():
    # p/q at token 0 is exactly 0.5 (p = (.25,.75), q = (.5,.5)); u within 1e-6 of it is flagged
    t = np.log(np.array([[[0.25, 0.75], [0.5, 0.5]]])).astype(np.float32)
    d = np.zeros((1, 1, 2), np.float32)
    ratio = (_softmax(t[0, 0]) / _softmax(d[0, 0]))[0]
    for du, flagged in ((3e-7, True), (-3e-7, True), (1e-4, False)):
        u = np.array([[[ratio + du, 0.5], [0.5, 0.5]]], np.float32)
        r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=np.zeros((1, 1), np.int32), uniforms=u))
        assert bool(r["near"][0] & oracle.NEAR_ACCEPT) == flagged


def test_step_composes_signals_controller_and_verification():
    rng = np.random.default_rng(15)
    B, G, V = 9, 4, 64
    t = rng.normal(0, 2, (B, G + 1, V)).astype(np.float32)
    d = (t[:, :G] + rng.normal(0, 0.5, (B, G, V))).astype(np.float32)
    tok = d.argmax(-1).astype(np.int32)
    gam = rng.integers(1, G + 1, B).astype(np.int32)
    u = rng.random((B, G + 1, 2)).astype(np.float32)
    comp = rng.integers(0, 2, (B, 2)).astype(np.float32)
    mlp = oracle.Mlp(rng.normal(0, 0.1, (16, 5)), rng.normal(0, 0.1, 16), rng.normal(0, 0.1, (4, 16)),
                     rng.normal(0, 0.1, 4))
    bt = oracle.Batch(draft=d, target=t, draft_tokens=tok, gamma=gam, uniforms=u, temperature_scalar=0.8)
    s = oracle.step(bt, comp, mlp)
    sig, ver = oracle.signals(bt), oracle.verify(bt)
    ctl = oracle.select_gamma(sig["feat"], comp, mlp)
    np.testing.assert_array_equal(s["H"], sig["H"])
    np.testing.assert_array_equal(s["feat"], sig["feat"])
    np.testing.assert_array_equal(s["n_accepted"], ver["n_accepted"])
    np.testing.assert_array_equal(s["out_tokens"], ver["out_tokens"])
    np.testing.assert_array_equal(s["scores"], ctl["scores"])
    np.testing.assert_array_equal(s["gamma_next"], ctl["gamma_next"])
    assert set(np.unique(s["gamma_next"])) <= {2, 4, 6, 8}


def test_vanishing_residual_is_drawn_exactly_and_flagged():
    # p and q agree to 1e-13 except on two far-tail tokens: the rejection of token 1 leaves a residual of
    # total mass about 6e-14, all of it on token 2.  The rule still fixes the draw (token 2, whatever u' is);
    # the row is marked, because weights held in fp32 cannot resolve such a residual.
    d = np.array([[[0.0, -30.0, -31.0]]], np.float32)
    t = np.array([[[0.0, -31.0, -30.0], [0.0, 0.0, 0.0]]], np.float32)
    for u2 in (0.0, 0.3, 0.999):
        u = np.array([[[0.9, u2], [0.5, 0.5]]], np.float32)
        r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=np.array([[1]], np.int32), uniforms=u))
        assert r["n_accepted"][0] == 0 and r["out_tokens"][0, 0] == 2
        assert r["near"][0] & oracle.NEAR_SMALL_RESIDUAL
    # the same shape of problem with an ordinary residual is not marked
    d2 = np.array([[[0.0, 1.0, -1.0]]], np.float32)
    t2 = np.array([[[0.0, -1.0, 1.0], [0.0, 0.0, 0.0]]], np.float32)
    r = oracle.verify(oracle.Batch(draft=d2, target=t2, draft_tokens=np.array([[1]], np.int32),
                                   uniforms=np.array([[[0.9, 0.5], [0.5, 0.5]]], np.float32)))
    assert r["n_accepted"][0] == 0 and r["out_tokens"][0, 0] == 2 and not (r["near"][0] & (oracle.NEAR_CDF | oracle.NEAR_SMALL_RESIDUAL))


def _four_token_case():
    """gamma = 2, V = 4.  Draft = uniform; the three target rows put their excess mass on different
    tokens, so that the residual of position i (and the bonus distribution of position 2) sits on a
    token of its own: position 0 -> token 1, position 1 -> token 2, position 2 -> token 3."""
    d = np.zeros((1, 2, 4), np.float32)
    t = np.full((1, 3, 4), 0.0, np.float32)
    t[0, 0, 1] = 3.0
    t[0, 1, 2] = 3.0
    t[0, 2, :] = [NEG, NEG, NEG, 0.0]          # bonus distribution: token 3 with probability 1
    return d, t


def test_second_uniform_is_taken_at_the_stop_position():
    # Token 0 has p/q = 4 p(0) < 1 at both drafted positions (p(0) = 1 / (3 + e^3) = 0.043, ratio 0.173).
    d, t = _four_token_case()
    p1 = _softmax(t[0, 1])
    assert 4 * p1[0] < 0.2
    tok = np.zeros((1, 2), np.int32)
    # residual of position 1 = max(0, p1 - 1/4): all of it on token 2; of position 0: all on token 1.
    # Accept position 0 (u = 0.01 < 0.173), reject position 1 (u = 0.9).  The second uniforms differ per
    # position; only u[b, 1, 1] may be consumed.  With a two-token residual the choice shows which one was.
    t2 = t.copy()
    t2[0, 1, :] = [0.0, 0.0, 2.0, 2.0]         # position 1: residual on tokens 2 and 3, equal halves
    u = np.zeros((1, 3, 2), np.float32)
    u[0, :, 0] = [0.01, 0.9, 0.5]
    for u11, want in ((0.25, 2), (0.75, 3)):
        for other in (0.25, 0.75):              # whatever the other positions' second uniforms say
            u[0, :, 1] = [other, u11, other]
            r = oracle.verify(oracle.Batch(draft=d, target=t2, draft_tokens=tok, uniforms=u))
            assert r["n_accepted"][0] == 1
            assert list(r["out_tokens"][0]) == [0, want, -1]
    # rejected at position 0 instead: the residual there is token 1 only, and u[b, 0, 1] is the one read
    u[0, :, 0] = [0.9, 0.01, 0.5]
    u[0, :, 1] = [0.5, 0.25, 0.75]
    r = oracle.verify(oracle.Batch(draft=d, target=t2, draft_tokens=tok, uniforms=u))
    assert r["n_accepted"][0] == 0 and list(r["out_tokens"][0]) == [1, -1, -1]


def test_bonus_draw_reads_the_second_uniform_of_position_gamma():
    # both drafted tokens accepted (u = 0.01); the bonus row splits its mass over tokens 1 and 3
    d, t = _four_token_case()
    t[0, 2, :] = [NEG, 0.0, NEG, 0.0]
    tok = np.zeros((1, 2), np.int32)
    u = np.zeros((1, 3, 2), np.float32)
    u[0, :, 0] = 0.01
    for u21, want in ((0.25, 1), (0.75, 3)):
        for other in (0.25, 0.75):
            u[0, :, 1] = [other, other, u21]
            r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, uniforms=u))
            assert r["n_accepted"][0] == 2 and list(r["out_tokens"][0]) == [0, 0, want]


def test_target_rows_behind_the_stop_position_are_not_part_of_the_step():
    # Sec. 3.1: the step emits the accepted prefix and one token at the first mismatch.  A NaN in a target
    # row behind the stop position changes nothing; at or before it, it flags the row.
    d, t = _four_token_case()
    tok = np.zeros((1, 2), np.int32)
    u = np.zeros((1, 3, 2), np.float32)
    u[0, :, 0] = [0.9, 0.01, 0.5]               # rejected at position 0
    u[0, :, 1] = 0.5
    clean = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, uniforms=u))
    assert clean["n_accepted"][0] == 0 and clean["row_status"][0] == 0
    for pos, flagged in ((0, True), (1, False), (2, False)):
        tt = t.copy()
        tt[0, pos, 3] = np.nan
        for T in (1.0, 0.0):                    # sampling rule and greedy rule (token 0 is never the argmax)
            r = oracle.verify(oracle.Batch(draft=d, target=tt, draft_tokens=tok, uniforms=u, temperature_scalar=T))
            assert (r["row_status"][0] == oracle.ROW_NONFINITE) == flagged, (pos, T)
            if not flagged:
                assert r["n_accepted"][0] == 0 and r["out_tokens"][0, 0] == 1
    # a non-finite *draft* row flags the row wherever it is: the signals use every drafted position
    dd = d.copy()
    dd[0, 1, 2] = np.inf
    r = oracle.verify(oracle.Batch(draft=dd, target=t, draft_tokens=tok, uniforms=u))
    assert r["row_status"][0] == oracle.ROW_NONFINITE and r["out_tokens"][0, 0] == -1
    # an out-of-range token ends the walk: a NaN behind it is not reached, one in front of it is
    tok2 = np.array([[0, 7]], np.int32)
    u[0, :, 0] = 0.01                           # position 0 accepted, position 1 cannot be tested
    for pos, want in ((2, oracle.ROW_BAD_TOKEN), (1, oracle.ROW_BAD_TOKEN | oracle.ROW_NONFINITE),
                      (0, oracle.ROW_BAD_TOKEN | oracle.ROW_NONFINITE)):
        tt = t.copy()
        tt[0, pos, 0] = np.nan
        r = oracle.verify(oracle.Batch(draft=d, target=tt, draft_tokens=tok2, uniforms=u))
        assert r["row_status"][0] == want, pos


def test_step_gives_flagged_rows_neutral_outputs():
    rng = np.random.default_rng(16)
    B, G, V = 5, 3, 24
    t = rng.normal(0, 1, (B, G + 1, V)).astype(np.float32)
    d = rng.normal(0, 1, (B, G, V)).astype(np.float32)
    tok = rng.integers(0, V, (B, G)).astype(np.int32)
    gam = np.array([3, 0, 3, 3, 3], np.int32)    # row 1: bad gamma
    tok[2, 1] = V + 3                            # row 2: bad token
    d[3, 2, 5] = np.nan                          # row 3: NaN in a draft row
    T = np.array([1, 1, 1, 1, np.nan], np.float32)  # row 4: bad temperature
    u = rng.random((B, G + 1, 2)).astype(np.float32)
    comp = np.zeros((B, 2), np.float32)
    mlp = oracle.Mlp(rng.normal(0, 0.1, (16, 5)), rng.normal(0, 0.1, 16), rng.normal(0, 0.1, (4, 16)),
                     rng.normal(0, 0.1, 4))
    s = oracle.step(oracle.Batch(draft=d, target=t, draft_tokens=tok, gamma=gam, temperature=T, uniforms=u), comp, mlp)
    assert list(s["row_status"]) == [0, oracle.ROW_BAD_GAMMA, oracle.ROW_BAD_TOKEN, oracle.ROW_NONFINITE,
                                     oracle.ROW_BAD_TEMPERATURE]
    for b in range(1, B):
        assert s["n_accepted"][b] == 0 and np.all(s["out_tokens"][b] == -1)
        assert s["gamma_next"][b] == 0 and np.all(s["scores"][b] == 0)
        assert np.all(s["H"][b] == 0) and np.all(s["C"][b] == 0) and np.all(s["feat"][b] == 0)
    # the healthy row is untouched by its neighbours
    assert s["gamma_next"][0] in (2, 4, 6, 8) and s["feat"][0, 0] > 0 and s["out_tokens"][0, s["n_accepted"][0]] >= 0


def test_residual_boundary_flags_relative_and_absolute():
    # q = (0.6, 0.2, 0.2), p = (0.59, 0.2, 0.21) up to float32 rounding: token 0 is rejected with probability
    # 1/60 and the residual, of mass W = 0.01, sits on token 2 alone, so every u' draws token 2 and no
    # boundary is near.  With p = (0.59, 0.205, 0.205) the residual splits into two halves of 0.005:
    # the boundary between tokens 1 and 2 lies at u' = 0.5.  A threshold 2e-5 * W away from it (2e-7 in units
    # of probability) is outside the window on the normalised CDF but inside the absolute one; a threshold
    # 0.1 * W away is outside both.
    d = np.log(np.array([[[0.6, 0.2, 0.2]]])).astype(np.float32)
    t = np.log(np.array([[[0.59, 0.205, 0.205], [1 / 3, 1 / 3, 1 / 3]]])).astype(np.float32)
    p, q = _softmax(t[0, 0]), _softmax(d[0, 0])
    w = np.maximum(0, p - q)
    W = w.sum()
    edge = w[1] / W
    tok = np.zeros((1, 1), np.int32)
    for du, want in ((2e-5, oracle.NEAR_CDF_ABS), (-2e-5, oracle.NEAR_CDF_ABS), (3e-7, oracle.NEAR_CDF), (0.1, 0)):
        u = np.array([[[0.999, edge + du], [0.5, 0.5]]], np.float32)
        r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, uniforms=u))
        assert r["n_accepted"][0] == 0 and r["out_tokens"][0, 0] == (2 if du > 0 else 1)
        assert r["near"][0] & (oracle.NEAR_CDF | oracle.NEAR_CDF_ABS) == want, (du, r["near"][0])
    # a bonus draw (weights are probabilities, W = 1) never carries the absolute flag alone
    u = np.array([[[0.0, 0.3], [0.5, 1 / 3 + 2e-5]]], np.float32)
    r = oracle.verify(oracle.Batch(draft=d, target=t, draft_tokens=tok, uniforms=u))
    assert r["n_accepted"][0] == 1 and not (r["near"][0] & oracle.NEAR_CDF_ABS)

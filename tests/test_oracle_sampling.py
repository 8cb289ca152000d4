"""Pins for the oracle's draft-side sampling (paper Sec. 3.1: the draft proposes gamma tokens):
inverse CDF of softmax(d / T) in vocabulary order, argmax at T = 0."""
import numpy as np
import scipy.special
import scipy.stats

import oracle


def test_inverse_cdf_against_numpy_searchsorted():
    rng = np.random.default_rng(0)
    B, G, V, T = 40, 3, 50, 0.7
    d = rng.normal(0, 2, (B, G, V)).astype(np.float32)
    u = rng.random((B, G)).astype(np.float32)
    out = oracle.sample_draft(oracle.Batch(draft=d, temperature_scalar=T, n_threads=2), u)
    q = scipy.special.softmax(d.astype(np.float64) / np.float64(np.float32(T)), axis=-1)
    cdf = np.cumsum(q, axis=-1)
    want = np.array([[np.searchsorted(cdf[b, i], u[b, i] * cdf[b, i, -1], side="right") for i in range(G)]
                     for b in range(B)])
    ok = (out["tokens"] == want) | ((out["near"] & oracle.NEAR_CDF) != 0)[:, None]
    assert ok.all() and (out["tokens"] == want).mean() > 0.99


def test_sampled_tokens_follow_the_draft_distribution():
    rng = np.random.default_rng(1)
    V, N, T = 8, 200_000, 1.3
    row = rng.normal(0, 1.5, V).astype(np.float32)
    d = np.broadcast_to(row, (N, 1, V))
    u = rng.random((N, 1)).astype(np.float32)
    tok = oracle.sample_draft(oracle.Batch(draft=d, temperature_scalar=T, n_threads=8), u)["tokens"][:, 0]
    q = scipy.special.softmax(row.astype(np.float64) / np.float64(np.float32(T)))
    assert scipy.stats.chisquare(np.bincount(tok, minlength=V), q * N).pvalue > 1e-4


def test_edges_u_zero_masked_tokens_greedy_and_ragged_gamma():
    d = np.full((3, 4, 6), -np.inf, np.float32)
    d[:, :, 2] = 1.0; d[:, :, 4] = 1.0                      # two tokens with equal mass, the rest masked
    gamma = np.array([4, 2, 4], np.int32)
    T = np.array([1.0, 1.0, 0.0], np.float32)
    u = np.array([[0.0, 0.49, 0.51, 0.999], [0.0, 0.9, 0.1, 0.1], [0.5, 0.5, 0.5, 0.5]], np.float32)
    out = oracle.sample_draft(oracle.Batch(draft=d, gamma=gamma, temperature=T), u)
    assert out["tokens"].tolist() == [[2, 2, 4, 4], [2, 4, -1, -1], [2, 2, 2, 2]]   # greedy: lowest index of the tie
    assert out["row_status"].tolist() == [0, 0, 0]
    d[1, 0, 3] = np.nan
    out = oracle.sample_draft(oracle.Batch(draft=d, gamma=gamma, temperature=T), u)
    assert out["row_status"].tolist() == [0, oracle.ROW_NONFINITE, 0] and out["tokens"][1].tolist() == [-1] * 4

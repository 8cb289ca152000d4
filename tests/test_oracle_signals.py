"""Pins for the oracle's draft signals (paper Sec. 4.2) against closed forms, invariants
and independent library routines.  None of these retypes the oracle's own formula: each
expected value is a closed form, or comes from scipy."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle

NEG = -np.inf


def _sig(draft, **kw):
    draft = np.asarray(draft)
    if draft.ndim == 1:
        draft = draft[None, None, :]
    elif draft.ndim == 2:
        draft = draft[None, :, :]
    return oracle.signals(oracle.Batch(draft=np.ascontiguousarray(draft), **kw))


def _bf16_bits(x):
    """float32 -> bf16 bit patterns by truncation-free construction: inputs must be exactly
    representable (tests only pass such values)."""
    x = np.asarray(x, np.float32)
    bits = x.view(np.uint32)
    assert np.all((bits & 0xFFFF) == 0), "value not exactly representable in bf16"
    return (bits >> 16).astype(np.uint16)


@pytest.mark.parametrize("V", [1, 2, 7, 1000, 32000])
@pytest.mark.parametrize("const", [0.0, -3.5, 11.0])
def test_uniform_row_has_entropy_log_v(V, const):
    r = _sig(np.full(V, const, np.float32))
    assert r["row_status"][0] == 0
    assert r["H"][0, 0] == pytest.approx(math.log(V), rel=1e-13, abs=1e-13)
    assert r["C"][0, 0] == pytest.approx(1.0 / V, rel=1e-13)


def test_bits_mode_is_log2_as_in_the_paper():
    # Sec. 4.2 writes H with log2: a uniform row over 1024 tokens has exactly 10 bits.
    r = _sig(np.zeros(1024, np.float32), entropy_in_bits=True)
    assert r["H"][0, 0] == pytest.approx(10.0, rel=1e-13)
    x = np.random.default_rng(0).normal(size=300).astype(np.float32)
    nats = _sig(x)["H"][0, 0]
    bits = _sig(x, entropy_in_bits=True)["H"][0, 0]
    assert bits == pytest.approx(nats / math.log(2.0), rel=1e-13)


@pytest.mark.parametrize("hot", [0, 5, 99])
def test_one_hot_row_has_zero_entropy_and_confidence_one(hot):
    x = np.full(100, NEG, np.float32)
    x[hot] = 2.5
    r = _sig(x)
    assert r["row_status"][0] == 0
    assert r["H"][0, 0] == 0.0
    assert r["C"][0, 0] == 1.0
    # finite but huge gap: everything else underflows
    y = np.zeros(100, np.float32)
    y[hot] = 2000.0
    r = _sig(y)
    assert r["H"][0, 0] == pytest.approx(0.0, abs=1e-300)
    assert r["C"][0, 0] == 1.0


@pytest.mark.parametrize("a", [-4.0, -0.5, 0.0, 0.25, 3.0, 30.0])
@pytest.mark.parametrize("T", [1.0, 0.5, 2.0])
def test_two_point_row_is_binary_entropy_of_sigmoid(a, T):
    x = np.full(64, NEG, np.float32)
    x[3], x[40] = a, 0.0
    r = _sig(x, temperature_scalar=T)
    s = 1.0 / (1.0 + math.exp(-a / T))
    s2 = 1.0 / (1.0 + math.exp(a / T))  # 1 - s without cancellation
    expect = -(s * math.log(s) + s2 * math.log(s2))
    assert r["H"][0, 0] == pytest.approx(expect, rel=1e-12, abs=1e-15)
    assert r["C"][0, 0] == pytest.approx(max(s, s2), rel=1e-13)


def test_subset_uniform_rows_and_step_aggregates():
    # position i is uniform over k_i tokens: H_i = ln k_i, c_i = 1/k_i, so the step signals
    # (mean, mean, max, min) are known in closed form.
    ks = [1, 4, 10, 25]
    V = 50
    d = np.full((1, 4, V), NEG, np.float32)
    for i, k in enumerate(ks):
        d[0, i, (np.arange(k) * 2) % V] = 1.25
    r = oracle.signals(oracle.Batch(draft=d))
    np.testing.assert_allclose(r["H"][0], [math.log(k) for k in ks], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(r["C"][0], [1.0 / k for k in ks], rtol=1e-13)
    f = r["feat"][0]
    assert f[0] == pytest.approx(sum(math.log(k) for k in ks) / 4, rel=1e-13)
    assert f[1] == pytest.approx(sum(1.0 / k for k in ks) / 4, rel=1e-13)
    assert f[2] == pytest.approx(math.log(25), rel=1e-13)
    assert f[3] == pytest.approx(1.0 / 25, rel=1e-13)


def test_ragged_gamma_ignores_unused_positions():
    ks = [2, 8, 5]
    V = 16
    d = np.full((2, 4, V), np.nan, np.float32)  # garbage beyond gamma must not be read
    for b, g in enumerate([3, 1]):
        for i in range(g):
            d[b, i] = NEG
            d[b, i, :ks[i]] = 0.0
    r = oracle.signals(oracle.Batch(draft=d, gamma=np.array([3, 1], np.int32)))
    assert list(r["row_status"]) == [0, 0]
    np.testing.assert_allclose(r["H"][0], [math.log(2), math.log(8), math.log(5), 0.0], rtol=1e-13)
    np.testing.assert_allclose(r["H"][1], [math.log(2), 0, 0, 0], rtol=1e-13)
    np.testing.assert_allclose(r["feat"][0], [(math.log(2) + math.log(8) + math.log(5)) / 3,
                                              (1 / 2 + 1 / 8 + 1 / 5) / 3, math.log(8), 1 / 8], rtol=1e-13)
    np.testing.assert_allclose(r["feat"][1], [math.log(2), 0.5, math.log(2), 0.5], rtol=1e-13)


def test_shift_invariance_and_bounds():
    rng = np.random.default_rng(1)
    x = rng.normal(0, 2, size=(1, 5, 4000)).astype(np.float32)
    a = oracle.signals(oracle.Batch(draft=x))
    # a shift that is exact in float32 for these magnitudes is not available in general, so
    # shift by a power of two on values pre-rounded to a coarse grid
    xg = np.round(x * 64) / 64
    a = oracle.signals(oracle.Batch(draft=xg.astype(np.float32)))
    b = oracle.signals(oracle.Batch(draft=(xg + 16.0).astype(np.float32)))
    np.testing.assert_allclose(a["H"], b["H"], rtol=1e-12)
    np.testing.assert_allclose(a["C"], b["C"], rtol=1e-12)
    f = a["feat"][0]
    assert 0.0 <= f[0] <= f[2] <= math.log(4000)
    assert 1.0 / 4000 <= f[3] <= f[1] <= 1.0


@pytest.mark.parametrize("T", [1.0, 0.8, 1.7])
def test_random_rows_match_scipy(T):
    rng = np.random.default_rng(2)
    x = rng.normal(0, 3, size=(3, 2, 5000)).astype(np.float32)
    r = oracle.signals(oracle.Batch(draft=x, temperature_scalar=T))
    # the temperature reaches the library as a float32 value
    q = scipy.special.softmax(x.astype(np.float64) / float(np.float32(T)), axis=-1)
    np.testing.assert_allclose(r["H"], scipy.stats.entropy(q, axis=-1), rtol=1e-11)
    np.testing.assert_allclose(r["C"], q.max(-1), rtol=1e-12)


def test_greedy_rows_use_unit_temperature_for_signals():
    rng = np.random.default_rng(3)
    x = rng.normal(0, 2, size=(2, 2, 300)).astype(np.float32)
    r = oracle.signals(oracle.Batch(draft=x, temperature=np.array([0.0, 1.0], np.float32)))
    q = scipy.special.softmax(x.astype(np.float64), axis=-1)
    np.testing.assert_allclose(r["H"], scipy.stats.entropy(q, axis=-1), rtol=1e-11)


def test_bf16_bit_patterns_decode_exactly():
    # 1.0 = 0x3F80, -2.0 = 0xC000, 0.15625 = 0x3E20 as bf16; the row (ln-free) closed form:
    # logits (ln-like exact values) 0 and 1 -> two-point sigmoid(1)
    x = np.full(8, NEG, np.float32)
    x[1], x[6] = 1.0, 0.0
    bits = _bf16_bits(x)
    assert bits[1] == 0x3F80 and bits[0] == 0xFF80
    r = _sig(bits)
    s = 1.0 / (1.0 + math.exp(-1.0))
    assert r["H"][0, 0] == pytest.approx(-(s * math.log(s) + (1 - s) * math.log(1 - s)), rel=1e-13)
    # same numbers through the float32 path
    r32 = _sig(x)
    assert r32["H"][0, 0] == r["H"][0, 0]


def test_strided_views_are_honoured():
    rng = np.random.default_rng(4)
    big = rng.normal(size=(3, 5, 40)).astype(np.float32)
    view = big[:, 1:4, :]
    a = oracle.signals(oracle.Batch(draft=view))
    b = oracle.signals(oracle.Batch(draft=np.ascontiguousarray(view)))
    np.testing.assert_array_equal(a["H"], b["H"])


def test_status_flags():
    x = np.zeros((5, 2, 10), np.float32)
    x[1, 0, 3] = np.nan
    x[2, 1, 0] = np.inf
    x[3, 0, :] = NEG
    r = oracle.signals(oracle.Batch(draft=x))
    assert list(r["row_status"]) == [0, oracle.ROW_NONFINITE, oracle.ROW_NONFINITE, oracle.ROW_NONFINITE, 0]
    assert np.all(r["H"][1:4] == 0) and np.all(r["feat"][1:4] == 0)
    r = oracle.signals(oracle.Batch(draft=x, gamma=np.array([0, 3, 1, 1, 2], np.int32)))
    assert r["row_status"][0] == oracle.ROW_BAD_GAMMA and r["row_status"][1] == oracle.ROW_BAD_GAMMA
    assert r["row_status"][2] == 0  # the +inf sits at position 1, unused with gamma = 1
    r = oracle.signals(oracle.Batch(draft=x, temperature=np.array([-1, 1, 1, 1, np.nan], np.float32)))
    assert r["row_status"][0] == oracle.ROW_BAD_TEMPERATURE
    assert r["row_status"][4] == oracle.ROW_BAD_TEMPERATURE


def _merge(a, b):
    """Merge rule for two partial softmax states (m, Z, S) of disjoint parts of one row, with
    Z = sum e^(x-m) and S = sum e^(x-m) (x-m): bring both to the common maximum and add."""
    m = max(a[0], b[0])
    out_z, out_s = 0.0, 0.0
    for (mk, zk, sk) in (a, b):
        f = math.exp(mk - m)
        out_z += zk * f
        out_s += f * (sk + (mk - m) * zk)
    return (m, out_z, out_s)


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_merging_random_partitions_reproduces_the_unsplit_signals(seed):
    # H = ln Z - S/Z and c = 1/Z from states merged over a random partition of the row must equal the
    # oracle's -sum q ln q and max q on the whole row (Sec. 4.2): this is the identity a split sweep rests on.
    rng = np.random.default_rng(seed)
    V, T = 5000 + 37 * seed, (1.0, 0.7, 1.3, 2.0)[seed]
    x = rng.normal(0, 3, V).astype(np.float32)
    x[rng.integers(0, V, 40)] = -np.inf            # masked tokens contribute nothing
    ref = _sig(x[None, None, :], temperature_scalar=T)
    cuts = np.sort(rng.choice(np.arange(1, V), size=int(rng.integers(1, 12)), replace=False))
    parts = np.split(x.astype(np.float64) / float(np.float32(T)), cuts)
    rng.shuffle(parts)                             # the merge is order-free
    state = None
    for part in parts:
        fin = part[np.isfinite(part)]
        if fin.size == 0:
            continue
        m = fin.max()
        e = np.exp(fin - m)
        st = (m, e.sum(), (e * (fin - m)).sum())
        state = st if state is None else _merge(state, st)
    m, Z, S = state
    assert math.log(Z) - S / Z == pytest.approx(ref["H"][0, 0], rel=1e-12, abs=1e-12)
    assert 1.0 / Z == pytest.approx(ref["C"][0, 0], rel=1e-12)

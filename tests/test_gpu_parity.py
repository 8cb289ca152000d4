"""Parity of the CUDA path (through the C ABI) against the CPU oracle on seeded inputs."""
import math

import numpy as np
import pytest
import scipy.stats
import torch

import oracle
import paper_2605_02888_b200 as speckv
from paper_2605_02888_b200 import binding, synth

from parity import close, compare_step, gpu_batch, mlp_pair, np_logits, oracle_batch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_both(w, step=0, gamma=None, attrs=None, rows=None, bits=False):
    s = synth.make_step(w, step, DEV, attrs=attrs, gamma=gamma)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = speckv.speckv_step(gpu_batch(s, entropy_in_bits=bits), s["comp"], gm)
    torch.cuda.synchronize()
    comp = s["comp"].cpu().numpy()
    ref = oracle.step(oracle_batch(s, rows=rows, entropy_in_bits=bits), comp if rows is None else comp[rows], om)
    return s, out, ref


# ---- tiny shapes: vocabulary sizes that are odd, below one vector, one chunk, several chunks ----
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("V", [8, 33, 257, 4099])
@pytest.mark.parametrize("B,G", [(1, 1), (3, 4), (2, 8)])
def test_tiny_shapes(dtype, V, B, G):
    w = synth.Workload("t", B=B, gamma_max=G, V=V, dtype=dtype, gamma_mode="ragged", temperature=0.9,
                       sigma_t=1.5, sigma_d=synth.SIGMA_LEVELS, seed=V + B)
    for step in range(3):
        s, out, ref = _run_both(w, step)
        compare_step(out, ref)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_mixed_greedy_and_sampling_rows_small(dtype):
    w = synth.Workload("t", B=40, gamma_max=6, V=5000, dtype=dtype, gamma_mode="ragged",
                       temperature_mode="mixed", sigma_d=(0.5,), frac_onehot=0.2, seed=3)
    s, out, ref = _run_both(w)
    rep = compare_step(out, ref)
    assert (s["temperature"] == 0).any() and (s["temperature"] > 0).any()


# ---- the five workloads at reduced batch, full vocabulary ----
def test_workload_tiny_fp32_v32000():
    w = synth.scaled(synth.WORKLOADS["tiny"], steps=6)
    for step in range(w.steps):
        s, out, ref = _run_both(w, step)
        compare_step(out, ref)


def test_workload_b64_closed_loop_bf16():
    w = synth.scaled(synth.WORKLOADS["b64"], B=16, steps=5)
    attrs = synth.row_attrs(w)
    gamma_gpu = attrs.gamma0.clone()
    emitted = 0
    for step in range(w.steps):
        s, out, ref = _run_both(w, step, gamma=gamma_gpu, attrs=attrs)
        rep = compare_step(out, ref)
        assert set(np.unique(ref["gamma_next"])) <= {2, 4, 6, 8}
        gamma_gpu = out["gamma_next"].clone()   # the controller's choice drives the next step
        emitted += int(out["n_accepted"].sum()) + w.B
    assert emitted >= w.B * w.steps


def test_workload_b256_ragged_bf16_v128256():
    w = synth.scaled(synth.WORKLOADS["b256"], B=32)
    s, out, ref = _run_both(w)
    rep = compare_step(out, ref)
    # rows whose draft equals the target accept every drafted token
    same = synth.row_attrs(w).identical.numpy()
    if same.any():
        assert np.all(out["n_accepted"].cpu().numpy()[same] == s["gamma"].cpu().numpy()[same])
    # side case: gamma uniform over 1..8
    w2 = synth.scaled(w, gamma_mode="ragged", B=16, seed=5)
    s, out, ref = _run_both(w2)
    compare_step(out, ref)


def test_workload_b512_mixed_fp32_v151936():
    w = synth.scaled(synth.WORKLOADS["b512_mixed"], B=24, frac_onehot=0.25)
    s, out, ref = _run_both(w)
    rep = compare_step(out, ref)
    hot = synth.row_attrs(w).onehot.numpy()
    assert hot.any()
    # confidence ~ 1 and entropy ~ 0 on the one-hot-peaked rows
    assert np.all(ref["feat"][hot][:, 3] > 0.999) and np.all(ref["feat"][hot][:, 0] < 1e-3)


def test_workload_b1024_groups_bf16():
    w = synth.scaled(synth.WORKLOADS["b1024_loop"], B=24, steps=3)
    attrs = synth.row_attrs(w)
    assert len(set(zip(attrs.cluster.tolist(), attrs.sigma_d.tolist()))) == 12
    gamma = attrs.gamma0.clone()
    for step in range(w.steps):
        s, out, ref = _run_both(w, step, gamma=gamma, attrs=attrs)
        compare_step(out, ref)
        gamma = out["gamma_next"].clone()


# ---- full batch of the benchmark workload, oracle on sampled rows ----
def test_b256_full_batch_sampled_rows():
    w = synth.WORKLOADS["b256"]
    rows = np.array([0, 1, 37, 64, 100, 101, 128, 199, 254, 255])
    s, out, ref = _run_both(w, rows=rows)
    rep = compare_step(out, ref, rows=rows)
    # properties that hold on every row
    n = out["n_accepted"].cpu().numpy(); g = s["gamma"].cpu().numpy()
    assert np.all((n >= 0) & (n <= g)) and np.all(out["row_status"].cpu().numpy() == 0)
    H = out["H"].cpu().numpy(); C = out["C"].cpu().numpy(); f = out["feat"].cpu().numpy()
    assert np.all(H >= 0) and np.all(H <= math.log(w.V) + 1e-4) and np.all(C <= 1.0 + 1e-6)
    assert np.all(f[:, 3] <= f[:, 1] + 1e-6) and np.all(f[:, 0] <= f[:, 2] + 1e-6)
    assert set(np.unique(out["gamma_next"].cpu().numpy())) <= {2, 4, 6, 8}


def test_b512_mixed_full_batch_sampled_rows():
    # fp32 logits at full size: the bulk-copy ring sweep in the configuration the benchmark can time
    w = synth.WORKLOADS["b512_mixed"]
    attrs = synth.row_attrs(w)
    greedy = np.nonzero(attrs.temperature.numpy() == 0)[0]
    hot = np.nonzero(attrs.onehot.numpy())[0]
    rows = np.unique(np.concatenate([[0, 1, 255, 256, 510, 511], greedy[:2], hot[:2]]))
    s, out, ref = _run_both(w, rows=rows, attrs=attrs)
    compare_step(out, ref, rows=rows)
    n = out["n_accepted"].cpu().numpy(); g = s["gamma"].cpu().numpy()
    assert np.all((n >= 0) & (n <= g)) and np.all(out["row_status"].cpu().numpy() == 0)
    H = out["H"].cpu().numpy(); C = out["C"].cpu().numpy()
    assert np.all(H >= 0) and np.all(H <= math.log(w.V) + 1e-4) and np.all(C <= 1.0 + 1e-6)
    ot = out["out_tokens"].cpu().numpy()
    assert np.all(ot[np.arange(w.B), n] >= 0) and np.all(ot[np.arange(w.B), n] < w.V)


def test_batches_beyond_the_ring_sweep_table_take_the_other_kernel():
    # more rows than the staged sweep's per-row tables hold: same results from the register-staged kernel
    w = synth.Workload("t", B=1100, gamma_max=2, V=512, dtype="fp32", gamma_mode="ragged", temperature=0.9,
                       sigma_d=synth.SIGMA_LEVELS, seed=12)
    rows = np.array([0, 1, 511, 1023, 1024, 1099])
    s, out, ref = _run_both(w, rows=rows)
    compare_step(out, ref, rows=rows)
    w2 = synth.scaled(w, B=1024)   # the largest batch the ring sweep takes
    s, out, ref = _run_both(w2, rows=rows[:4])
    compare_step(out, ref, rows=rows[:4])


# ---- separate entry points ----
def test_signals_verify_and_controller_entry_points_agree_with_step():
    w = synth.Workload("t", B=12, gamma_max=5, V=9000, dtype="bf16", gamma_mode="ragged", temperature=0.7,
                       sigma_d=synth.SIGMA_LEVELS, seed=9)
    s = synth.make_step(w, 0, DEV)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    bt = gpu_batch(s)
    st = {k: v.clone() for k, v in speckv.speckv_step(bt, s["comp"], gm).items()}
    sig = speckv.speckv_signals(bt)
    ver = speckv.speckv_verify(bt)
    ctl = speckv.speckv_select_gamma(sig["feat"], s["comp"], gm)
    torch.cuda.synchronize()
    # the entry points cut the logit stream differently, so floats agree to rounding, not bit for bit
    for k in ("H", "C", "feat"):
        close(sig[k].cpu().numpy(), st[k].cpu().numpy(), k, rtol=2e-6, atol=1e-7)
    for k in ("n_accepted", "out_tokens"):
        assert torch.equal(ver[k], st[k]), k
    assert torch.equal(ctl["gamma_next"], st["gamma_next"])
    close(ctl["scores"].cpu().numpy(), st["scores"].cpu().numpy(), "scores", rtol=1e-6)
    ref = oracle.signals(oracle_batch(s))
    close(sig["H"].cpu().numpy(), ref["H"], "H")
    # bits mode (the paper's log2)
    sigb = speckv.speckv_signals(gpu_batch(s, entropy_in_bits=True))
    refb = oracle.signals(oracle_batch(s, entropy_in_bits=True))
    close(sigb["H"].cpu().numpy(), refb["H"], "H bits")
    close(sigb["feat"].cpu().numpy(), refb["feat"], "feat bits")


def test_paper_form_controller_layout():
    rng = np.random.default_rng(0)
    feat = torch.tensor(np.abs(rng.normal(size=(100, 4))), dtype=torch.float32, device=DEV)
    comp = torch.tensor(rng.integers(0, 3, (100, 1)), dtype=torch.float32, device=DEV)
    w = {k: torch.tensor(rng.normal(0, 0.1, shp), dtype=torch.float32, device=DEV)
         for k, shp in (("W1", (16, 5)), ("b1", (16,)), ("W2", (4, 16)), ("b2", (4,)))}
    for kw in (dict(feature_layout=1), dict(feature_layout=1, score_transform=1), dict()):
        gm, om = mlp_pair(w, **kw)
        c = comp if kw.get("feature_layout") else torch.cat([comp, comp], 1).clamp(max=1)
        out = speckv.speckv_select_gamma(feat, c, gm)
        ref = oracle.select_gamma(feat.cpu().numpy().astype(np.float64), c.cpu().numpy(), om)
        close(out["scores"].cpu().numpy(), ref["scores"], "scores")
        bad = out["gamma_next"].cpu().numpy() != ref["gamma_next"]
        assert not (bad & ((ref["near"] & oracle.NEAR_GAMMA) == 0)).any()


def test_paper_form_predictor_per_candidate_gamma():
    # Sec. 4.3 as printed: one predictor f(x, gamma) -> a_hat, evaluated for every candidate gamma
    rng = np.random.default_rng(1)
    feat = torch.tensor(np.abs(rng.normal(size=(200, 4))), dtype=torch.float32, device=DEV)
    comp = torch.tensor(rng.integers(0, 3, (200, 1)), dtype=torch.float32, device=DEV)
    t = lambda a: torch.tensor(a, dtype=torch.float32, device=DEV)
    mlp16 = dict(W1=t(rng.normal(0, 0.3, (16, 6))), b1=t(rng.normal(0, 0.3, 16)), W2=t(rng.normal(0, 0.3, (1, 16))),
                 b2=t(rng.normal(0, 0.1, 1)))
    ridge = dict(W1=torch.zeros(0, 6, device=DEV), b1=torch.zeros(0, device=DEV), W2=t(rng.normal(0, 0.2, (1, 6))),
                 b2=t([0.4]))
    for w in (mlp16, ridge):
        for kw in (dict(feature_layout=2), dict(feature_layout=2, score_transform=1)):
            gm, om = mlp_pair(w, **kw)
            out = speckv.speckv_select_gamma(feat, comp, gm)
            ref = oracle.select_gamma(feat.cpu().numpy().astype(np.float64), comp.cpu().numpy(), om)
            assert out["scores"].shape == (200, 4)
            close(out["scores"].cpu().numpy(), ref["scores"], "scores", atol=2e-7)
            bad = out["gamma_next"].cpu().numpy() != ref["gamma_next"]
            assert not (bad & ((ref["near"] & oracle.NEAR_GAMMA) == 0)).any()
    # and inside the fused step
    wl = synth.Workload("t", B=10, gamma_max=4, V=3000, dtype="fp32", gamma_mode="ragged", sigma_d=(0.5,), seed=2)
    s = synth.make_step(wl, 0, DEV)
    gm, om = mlp_pair(mlp16, feature_layout=2)
    comp1 = s["comp"][:, :1].contiguous()
    out = speckv.speckv_step(gpu_batch(s), comp1, gm)
    ref = oracle.step(oracle_batch(s), comp1.cpu().numpy(), om)
    compare_step(out, ref)


# ---- draft-side sampling ----
@pytest.mark.parametrize("dtype,V", [("bf16", 128256), ("fp32", 4099), ("bf16", 33)])
def test_sample_draft_against_oracle(dtype, V):
    w = synth.Workload("t", B=20, gamma_max=5, V=V, dtype=dtype, gamma_mode="ragged", temperature_mode="mixed",
                       sigma_d=(0.5,), seed=31)
    s = synth.make_step(w, 0, DEV)
    u = torch.rand(w.B, w.gamma_max, device=DEV)
    u[0, 0] = 0.0
    out = speckv.speckv_sample_draft(gpu_batch(s), u)
    ref = oracle.sample_draft(oracle_batch(s), u.cpu().numpy())
    tok = out["tokens"].cpu().numpy()
    np.testing.assert_array_equal(out["row_status"].cpu().numpy(), ref["row_status"])
    bad = (tok != ref["tokens"]).any(1)
    assert not (bad & ((ref["near"] & oracle.NEAR_CDF) == 0)).any()
    g = s["gamma"].cpu().numpy()
    cols = np.arange(w.gamma_max)[None, :]
    assert np.all(tok[cols >= g[:, None]] == -1) and np.all(tok[cols < g[:, None]] >= 0)
    assert (s["temperature"] == 0).any() and (s["temperature"] > 0).any()


def test_sample_draft_very_long_rows_take_the_two_pass_form():
    # more chunks per row than the one-pass kernel stages: normaliser sweep, then the weights
    w = synth.Workload("t", B=3, gamma_max=2, V=600_000, dtype="fp32", gamma_mode="fixed", gamma_fixed=2,
                       temperature_mode="mixed", sigma_d=(0.5,), seed=33)
    s = synth.make_step(w, 0, DEV)
    u = torch.rand(w.B, w.gamma_max, device=DEV)
    out = speckv.speckv_sample_draft(gpu_batch(s), u)
    ref = oracle.sample_draft(oracle_batch(s), u.cpu().numpy())
    np.testing.assert_array_equal(out["row_status"].cpu().numpy(), ref["row_status"])
    bad = (out["tokens"].cpu().numpy() != ref["tokens"]).any(1)
    assert not (bad & ((ref["near"] & oracle.NEAR_CDF) == 0)).any()


def test_sample_draft_distribution_and_flags():
    rng = np.random.default_rng(8)
    V, N, T = 8, 200_000, 0.9
    row = torch.tensor(rng.normal(0, 1.4, (1, V)), dtype=torch.float32, device=DEV)
    u = torch.rand(N, 1, device=DEV)
    out = speckv.speckv_sample_draft(speckv.Batch(draft_logits=row[None].expand(N, 1, V), temperature_scalar=T), u)
    q = torch.softmax(row[0].double() / float(np.float32(T)), -1).cpu().numpy()
    cnt = np.bincount(out["tokens"].cpu().numpy()[:, 0], minlength=V)
    assert scipy.stats.chisquare(cnt, q * N).pvalue > 1e-4
    d = torch.zeros(3, 2, 64, device=DEV)
    d[1, 1, 7] = float("nan")
    gam = torch.tensor([2, 2, 0], dtype=torch.int32, device=DEV)
    out = speckv.speckv_sample_draft(speckv.Batch(draft_logits=d, gamma=gam), torch.rand(3, 2, device=DEV))
    assert out["row_status"].tolist() == [0, 4, 1]
    assert out["tokens"][1:].flatten().tolist() == [-1] * 4 and (out["tokens"][0] >= 0).all()


# ---- edge cases ----
def _small(dtype="fp32", B=6, G=3, V=600, seed=0):
    w = synth.Workload("e", B=B, gamma_max=G, V=V, dtype=dtype, gamma_mode="fixed", gamma_fixed=G,
                       temperature=1.0, sigma_d=(0.5,), seed=seed)
    return w, synth.make_step(w, 0, DEV)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_row_status_flags(dtype):
    w, s = _small(dtype, B=8)
    s["target"][1, 0, 17] = float("nan")       # position 0 is read whatever happens behind it
    s["draft"][2, 0, 5] = float("inf")
    s["draft"][3, 1, :] = float("-inf")
    s["draft_tokens"][4, 1] = w.V
    s["gamma"][5] = 0
    s["temperature"][6] = -1.0
    s["target"][7, 0, :] = float("-inf")
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
    ref = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
    assert list(ref["row_status"]) == [0, 4, 4, 4, 2, 1, 8, 4]
    compare_step(out, ref)
    o = {k: v.cpu().numpy() for k, v in out.items()}
    assert np.all(o["n_accepted"][1:] == 0) and np.all(o["out_tokens"][1:] == -1)
    assert np.all(o["gamma_next"][1:] == 0) and np.all(o["H"][1:] == 0) and np.all(o["scores"][1:] == 0)
    # target rows behind the stop position are not part of the step (Sec. 3.1): a NaN there flags nothing,
    # a NaN at the stop position does
    n0 = int(ref["n_accepted"][0])
    if n0 < w.gamma_max:
        s["target"][0, n0 + 1:, 3] = float("nan")
        out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
        ref2 = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
        assert ref2["row_status"][0] == 0 and ref2["n_accepted"][0] == n0
        compare_step(out, ref2)
    s["target"][0, n0, 3] = float("nan")
    out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
    ref3 = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
    assert ref3["row_status"][0] == 4
    compare_step(out, ref3)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_masked_vocabulary_minus_inf(dtype):
    w, s = _small(dtype, B=5, V=3000)
    mask = torch.rand(w.V, device=DEV) < 0.6
    s["draft"][:, :, mask] = float("-inf")
    s["target"][:, :, mask] = float("-inf")
    keep = (~mask).nonzero().flatten()
    s["draft_tokens"] = keep[torch.randint(0, len(keep), s["draft_tokens"].shape, device=DEV)].to(torch.int32)
    # one row drafts a token the target masks out: must be rejected
    s["target"][0, 0, int(s["draft_tokens"][0, 0])] = float("-inf")
    # a whole leading region of -inf (first vectors of every thread)
    s["draft"][1, :, :2100] = float("-inf")
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
    ref = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
    assert ref["n_accepted"][0] == 0 and np.all(ref["row_status"] == 0)
    compare_step(out, ref)


def test_closed_forms_on_the_gpu():
    V = 128256
    d = torch.zeros(3, 2, V, device=DEV)
    d[1, :, :] = float("-inf"); d[1, 0, 77] = 3.0; d[1, 1, V - 1] = -2.0   # one-hot rows
    d[2, 0, 5] = 40.0                                                       # gap 40 over a flat tail
    out = speckv.speckv_signals(speckv.Batch(draft_logits=d))
    H = out["H"].cpu().numpy(); C = out["C"].cpu().numpy()
    assert H[0, 0] == pytest.approx(math.log(V), rel=1e-6) and C[0, 0] == pytest.approx(1 / V, rel=1e-6)
    assert H[1, 0] == 0.0 and H[1, 1] == 0.0 and C[1, 0] == 1.0
    eps = (V - 1) * math.exp(-40.0)
    assert H[2, 0] == pytest.approx(math.log1p(eps) + 40.0 * eps / (1 + eps), rel=1e-5)
    outb = speckv.speckv_signals(speckv.Batch(draft_logits=d, entropy_in_bits=True))
    assert outb["H"].cpu().numpy()[0, 0] == pytest.approx(math.log2(V), rel=1e-6)


def test_identical_logits_accept_everything_and_extreme_uniforms():
    w, s = _small("bf16", B=7, G=6, V=2048)
    s["draft"] = s["target"][:, :w.gamma_max].clone()
    s["uniforms"][0] = 0.0
    s["uniforms"][1] = 1.0 - 2 ** -24
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
    ref = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
    assert np.all(ref["n_accepted"] == w.gamma_max)
    compare_step(out, ref)


def test_gamma_max_16_and_strided_views():
    w = synth.Workload("e", B=3, gamma_max=16, V=1000, dtype="bf16", gamma_mode="ragged", sigma_d=(0.3,), seed=4)
    s = synth.make_step(w, 0, DEV)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
    ref = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
    compare_step(out, ref)
    # logits that live in a wider buffer: vocabulary padded to 1024, rows not adjacent
    padded_t = torch.full((w.B, w.gamma_max + 1, 1024), 7.0, dtype=torch.bfloat16, device=DEV)
    padded_d = torch.full((w.B, w.gamma_max + 3, 1024), 7.0, dtype=torch.bfloat16, device=DEV)
    padded_t[:, :, :1000] = s["target"]; padded_d[:, 1:w.gamma_max + 1, :1000] = s["draft"]
    s2 = dict(s); s2["target"] = padded_t[:, :, :1000]; s2["draft"] = padded_d[:, 1:w.gamma_max + 1, :1000]
    out2 = speckv.speckv_step(gpu_batch(s2), s["comp"], gm)
    for k in out:
        assert torch.equal(out[k], out2[k]), k
    # misaligned base (element offset 1) takes the element-wise path and gives the same results
    off_t = torch.zeros(w.B * (w.gamma_max + 1) * 1000 + 1, dtype=torch.bfloat16, device=DEV)
    off_t[1:] = s["target"].flatten()
    s3 = dict(s); s3["target"] = off_t[1:].view(w.B, w.gamma_max + 1, 1000)
    out3 = speckv.speckv_step(gpu_batch(s3), s["comp"], gm)
    compare_step(out3, ref)


def test_ring_sweep_with_padded_rows_and_ragged_ends_fp32():
    # fp32 logits in a wider buffer: rows 16-byte aligned but not adjacent, V not a multiple of a block
    # (the ring sweep is chosen for fp32 batches of 384 to 1024 rows)
    w = synth.Workload("e", B=390, gamma_max=6, V=5004, dtype="fp32", gamma_mode="ragged", temperature_mode="mixed",
                       sigma_d=(0.4,), frac_onehot=0.05, frac_identical=0.05, seed=14)
    s = synth.make_step(w, 0, DEV)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    ref = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
    out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
    compare_step(out, ref)
    pt = torch.full((w.B, w.gamma_max + 2, 5120), 3.0, device=DEV)
    pd = torch.full((w.B, w.gamma_max + 1, 5120), 3.0, device=DEV)
    pt[:, 1:w.gamma_max + 2, :w.V] = s["target"]; pd[:, :w.gamma_max, :w.V] = s["draft"]
    s2 = dict(s); s2["target"] = pt[:, 1:w.gamma_max + 2, :w.V]; s2["draft"] = pd[:, :w.gamma_max, :w.V]
    out2 = speckv.speckv_step(gpu_batch(s2), s["comp"], gm)
    for k in out:
        assert torch.equal(out[k], out2[k]), k
    # an element offset of one breaks the 16-byte alignment: the register-staged kernel's element-wise path
    flat = torch.zeros(s["target"].numel() + 1, device=DEV)
    flat[1:] = s["target"].flatten()
    s3 = dict(s); s3["target"] = flat[1:].view_as(s["target"])
    compare_step(speckv.speckv_step(gpu_batch(s3), s["comp"], gm), ref)
    # the same aligned batch through the sliced sweep, asked for by flag
    compare_step(speckv.speckv_step(gpu_batch(s, flags=binding.SCHEDULE_SLICED), s["comp"], gm), ref)


@pytest.mark.parametrize("name,B,V", [("b256", 16, 128256), ("b512_mixed", 16, 151936), ("b512_mixed", 400, 8000)])
def test_results_are_deterministic(name, B, V):
    w = synth.scaled(synth.WORKLOADS[name], B=B, V=V)   # 400 fp32 rows: the ring sweep
    s = synth.make_step(w, 0, DEV)
    gm, _ = mlp_pair(synth.make_mlp(w, DEV))
    a = {k: v.clone() for k, v in speckv.speckv_step(gpu_batch(s), s["comp"], gm).items()}
    for _ in range(3):
        b = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
        for k in a:
            assert torch.equal(a[k].view(torch.int32) if a[k].dtype == torch.float32 else a[k],
                               b[k].view(torch.int32) if b[k].dtype == torch.float32 else b[k]), k


def test_full_size_step_repeats_bit_for_bit_with_one_workspace():
    # the fresh tokens are drawn by CTAs that wait for a row's completion flag while other rows are still
    # being swept: a missed ordering would show as a run that differs, or as a row flagged TIMEOUT
    w = synth.WORKLOADS["b256"]
    s = synth.make_step(w, 0, DEV)
    gm, _ = mlp_pair(synth.make_mlp(w, DEV))
    bt = gpu_batch(s)
    out = speckv.StepOutputs.allocate(bt, gm.n_out)
    first = {k: v.clone() for k, v in speckv.speckv_step(bt, s["comp"], gm, out=out).items()}
    assert int(first["row_status"].abs().sum()) == 0
    assert int((first["out_tokens"][torch.arange(w.B), first["n_accepted"].long()] < 0).sum()) == 0
    for _ in range(40):
        again = speckv.speckv_step(bt, s["comp"], gm, out=out)
        for k, v in first.items():
            assert torch.equal(v.view(torch.int32) if v.dtype == torch.float32 else v,
                               again[k].view(torch.int32) if again[k].dtype == torch.float32 else again[k]), k


def _same_bits(a, b):
    for k, v in a.items():
        assert torch.equal(v.view(torch.int32) if v.dtype == torch.float32 else v,
                           b[k].view(torch.int32) if b[k].dtype == torch.float32 else b[k]), k


@pytest.mark.parametrize("B,V", [(256, 128256), (300, 8200), (24, 50264)])
def test_target_rows_behind_a_rejection_are_skipped_without_changing_anything(B, V):
    # the sliced sweep leaves target rows unread when a rejection at position 0 or 1 is known before their CTAs
    # start (a matter of timing, so the full-size batch, where it does happen, a batch of short rows and a small
    # batch, where it mostly does not): with and without the skipping the outputs are the same bits; and they
    # stay the same when every target row behind a row's stop position is overwritten with NaN, read or not
    w = synth.scaled(synth.WORKLOADS["b256"], B=B, V=V)
    s = synth.make_step(w, 0, DEV)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    skip = {k: v.clone() for k, v in speckv.speckv_step(gpu_batch(s), s["comp"], gm).items()}
    full = {k: v.clone() for k, v in speckv.speckv_step(gpu_batch(s, flags=binding.READ_ALL_TARGET_ROWS), s["comp"], gm).items()}
    _same_bits(skip, full)
    assert int(skip["row_status"].abs().sum()) == 0
    rows = np.arange(0, B, max(1, B // 24))
    ref = oracle.step(oracle_batch(s, rows=rows), s["comp"].cpu().numpy()[rows], om)
    compare_step(skip, ref, rows=rows)
    n, g = skip["n_accepted"].long(), s["gamma"].long()
    pos = torch.arange(w.gamma_max + 1, device=DEV)[None, :]
    behind = (pos > n[:, None]) & (pos <= g[:, None])
    assert int(behind.sum()) > 0
    s["target"][behind] = float("nan")
    for flags in (0, binding.READ_ALL_TARGET_ROWS):
        for _ in range(3):
            _same_bits(skip, speckv.speckv_step(gpu_batch(s, flags=flags), s["comp"], gm))


@pytest.mark.parametrize("name,B,V,flags", [("b256", 64, 32000, 0), ("b512_mixed", 400, 8000, 0), ("b512_mixed", 32, 8000, 0),
                                            ("b512_mixed", 400, 8000, 4)])
def test_step_can_be_captured_in_a_cuda_graph(name, B, V, flags):
    # the library only enqueues work on the caller's stream (no allocation, no synchronisation), so a step
    # can be recorded once and replayed: single-launch path, ring sweep + dependent resample kernel, fp32 fallback,
    # and the sliced sweep asked for by flag for a batch that would take the ring (flags = 4, SPECKV_SCHEDULE_SLICED)
    w = synth.scaled(synth.WORKLOADS[name], B=B, V=V)
    s = synth.make_step(w, 0, DEV)
    gm, _ = mlp_pair(synth.make_mlp(w, DEV))
    bt = gpu_batch(s, flags=flags)
    out = speckv.StepOutputs.allocate(bt, gm.n_out)
    direct = {k: v.clone() for k, v in speckv.speckv_step(bt, s["comp"], gm, out=out).items()}
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        speckv.speckv_step(bt, s["comp"], gm, out=out)          # warm-up on the capturing stream
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            speckv.speckv_step(bt, s["comp"], gm, out=out)
    for _ in range(3):
        for v in out.as_dict().values():
            v.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for k, v in direct.items():
            assert torch.equal(v.view(torch.int32) if v.dtype == torch.float32 else v,
                               out.as_dict()[k].view(torch.int32) if v.dtype == torch.float32 else out.as_dict()[k]), k


def test_steps_overlapping_on_several_streams_match_their_serial_results():
    # each call has its own workspace and outputs; the kernels of different calls share the SMs, among them
    # CTAs that wait for a flag of their own grid and the persistent ring sweep
    cfgs = [synth.scaled(synth.WORKLOADS["b256"], B=200), synth.scaled(synth.WORKLOADS["b512_mixed"], B=64, V=32000),
            synth.scaled(synth.WORKLOADS["b1024_loop"], B=300, V=50000), synth.scaled(synth.WORKLOADS["b512_mixed"], B=400, V=16000)]
    items = []
    for w in cfgs:
        s = synth.make_step(w, 0, DEV)
        gm, _ = mlp_pair(synth.make_mlp(w, DEV))
        bt = gpu_batch(s)
        out = speckv.StepOutputs.allocate(bt, gm.n_out)
        serial = {k: v.clone() for k, v in speckv.speckv_step(bt, s["comp"], gm, out=out).items()}
        items.append((s, gm, bt, out, serial))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in items]
    for _ in range(12):
        for st, (s, gm, bt, out, serial) in zip(streams, items):
            with torch.cuda.stream(st):
                for v in out.as_dict().values():
                    v.zero_()
                speckv.speckv_step(bt, s["comp"], gm, out=out)
        torch.cuda.synchronize()
        for s, gm, bt, out, serial in items:
            for k, v in serial.items():
                a = out.as_dict()[k]
                assert torch.equal(v.view(torch.int32) if v.dtype == torch.float32 else v,
                                   a.view(torch.int32) if a.dtype == torch.float32 else a), k


def test_empty_batch_and_argument_errors():
    d = torch.zeros(0, 4, 100, device=DEV)
    out = speckv.speckv_signals(speckv.Batch(draft_logits=d))
    assert out["H"].shape == (0, 4)
    w, s = _small()
    bt = gpu_batch(s)
    o = speckv.StepOutputs.allocate(bt)
    # the binding refuses buffers of the wrong size, shape or type before anything is launched
    short = speckv.StepOutputs.allocate(bt)
    short.workspace = short.workspace[:256]
    with pytest.raises(ValueError, match="workspace"):
        speckv.speckv_verify(bt, out=short)
    bad = speckv.StepOutputs.allocate(bt)
    bad.out_tokens = bad.out_tokens[:, :-1].contiguous()
    with pytest.raises(ValueError, match="out_tokens"):
        speckv.speckv_verify(bt, out=bad)
    bad = speckv.StepOutputs.allocate(bt)
    bad.H = bad.H.double()
    with pytest.raises(TypeError, match="H"):
        speckv.speckv_signals(bt, out=bad)
    gm, _ = mlp_pair(synth.make_mlp(w, DEV))
    with pytest.raises(ValueError, match="comp"):
        speckv.speckv_step(bt, s["comp"][:, :1].contiguous(), gm)
    with pytest.raises(ValueError, match="uniforms"):
        speckv.Batch(draft_logits=s["draft"], target_logits=s["target"], draft_tokens=s["draft_tokens"],
                     uniforms=s["uniforms"][:, :-1].contiguous())._c()
    # the library's own check of a short workspace, through the C ABI
    n = o.workspace.numel()
    rc = speckv.load_library().speckv_verify(__import__("ctypes").byref(bt._c()), o.n_accepted.data_ptr(), o.out_tokens.data_ptr(),
                                             o.row_status.data_ptr(), o.workspace.data_ptr(), n - 1, None)
    assert rc == 3


# ---- statistical properties of the CUDA path itself ----
def test_gpu_emitted_tokens_follow_target_distribution():
    # V = 8, gamma = 3, 250k trials sharing one set of logits (row stride 0)
    rng = np.random.default_rng(5)
    V, G, N, T = 8, 3, 250_000, 0.9
    tl = torch.tensor(rng.normal(0, 1.2, (G + 1, V)), dtype=torch.float32, device=DEV)
    dl = (tl[:G] + torch.tensor(rng.normal(0, 0.8, (G, V)), dtype=torch.float32, device=DEV)).contiguous()
    p = torch.softmax(tl.double() / float(np.float32(T)), -1).cpu().numpy()
    q = torch.softmax(dl.double() / float(np.float32(T)), -1)
    tok = torch.stack([torch.multinomial(q[i], N, replacement=True) for i in range(G)], 1).to(torch.int32)
    u = torch.rand(N, G + 1, 2, device=DEV)
    bt = speckv.Batch(draft_logits=dl[None].expand(N, G, V), target_logits=tl[None].expand(N, G + 1, V),
                      draft_tokens=tok.contiguous(), uniforms=u, temperature_scalar=T)
    out = speckv.speckv_verify(bt)
    n = out["n_accepted"].cpu().numpy(); ot = out["out_tokens"].cpu().numpy()
    assert np.all(out["row_status"].cpu().numpy() == 0)
    for i in range(G + 1):
        reached = n >= i
        cnt = np.bincount(ot[reached, i], minlength=V)
        assert scipy.stats.chisquare(cnt, p[i] * reached.sum()).pvalue > 1e-4
    # same inputs through the oracle: bit-exact apart from flagged near-ties
    ref = oracle.verify(oracle.Batch(draft=np.broadcast_to(dl.cpu().numpy()[None], (N, G, V)),
                                     target=np.broadcast_to(tl.cpu().numpy()[None], (N, G + 1, V)),
                                     draft_tokens=tok.cpu().numpy(), uniforms=u.cpu().numpy(),
                                     temperature_scalar=T, n_threads=8))
    bad = (ot != ref["out_tokens"]).any(1) | (n != ref["n_accepted"])
    assert not (bad & (ref["near"] == 0)).any()
    assert bad.sum() <= 20

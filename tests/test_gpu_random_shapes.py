"""Seeded sweep over batch / gamma / vocabulary shapes, dtypes and row mixes: the fused step (three times,
to catch an ordering that only sometimes holds), the vocabulary-sharded step and the draft sampling
against the oracle."""
import random

import numpy as np
import pytest
import torch

import oracle
import paper_2605_02888_b200 as speckv
from paper_2605_02888_b200 import binding, synth, vocab_shard

from parity import compare_step, gpu_batch, mlp_pair, oracle_batch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes(seed):
    rnd = random.Random(seed)
    for _ in range(30):
        B = rnd.choice([1, 2, 3, 7, 16, 33, 64, 65, 100, 257, 390, 500, 1030])
        G = rnd.choice([1, 2, 3, 4, 5, 8, 11, 16])
        V = rnd.choice([8, 31, 256, 257, 1000, 4099, 8192, 20000, 50257])
        if B * G * V > 3e8:
            V = 1000
        dtype = rnd.choice(["bf16", "fp32"])
        w = synth.Workload("s", B=B, gamma_max=G, V=V, dtype=dtype, gamma_mode=rnd.choice(["ragged", "choices", "fixed"]),
                           gamma_fixed=G, temperature_mode=rnd.choice(["mixed", "scalar"]),
                           temperature=rnd.choice([0.5, 1.0, 1.7]), sigma_d=synth.SIGMA_LEVELS,
                           frac_onehot=rnd.choice([0, 0.1]), frac_identical=rnd.choice([0, 0.1]), seed=rnd.randrange(1000))
        s = synth.make_step(w, rnd.randrange(5), DEV)
        gm, om = mlp_pair(synth.make_mlp(w, DEV))
        ref = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
        for _rep in range(3):
            out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
            torch.cuda.synchronize()
            compare_step(out, ref)
        for flags in (binding.SCHEDULE_SLICED, binding.READ_ALL_TARGET_ROWS):   # the other kernel choice; every target row read
            out = speckv.speckv_step(gpu_batch(s, flags=flags), s["comp"], gm)
            torch.cuda.synchronize()
            compare_step(out, ref)
        if V >= 64 and rnd.random() < 0.4:
            n_shards = rnd.choice([2, 3, 4])
            out = vocab_shard.step_emulated(gpu_batch(s), n_shards, s["comp"], gm)
            torch.cuda.synchronize()
            compare_step(out, ref)
        u = torch.rand(B, G, device=DEV)
        got = speckv.speckv_sample_draft(gpu_batch(s), u)
        want = oracle.sample_draft(oracle_batch(s), u.cpu().numpy())
        np.testing.assert_array_equal(got["row_status"].cpu().numpy(), want["row_status"])
        bad = (got["tokens"].cpu().numpy() != want["tokens"]).any(1)
        assert not (bad & ((want["near"] & oracle.NEAR_CDF) == 0)).any(), (B, G, V, dtype)


@pytest.mark.parametrize("seed", [21])
def test_random_edge_inputs(seed):
    """Masked vocabularies (-inf in the same columns of draft and target), temperatures changed after the
    draft tokens were drawn (1e-6 .. 50: tokens of vanishing probability under both models), planted NaN,
    +inf, all -inf rows and zero uniforms."""
    rnd = random.Random(seed)
    for it in range(40):
        B = rnd.choice([4, 20, 70, 300, 400])
        G = rnd.choice([2, 4, 8])
        V = rnd.choice([257, 1000, 4099, 8192])
        dtype = rnd.choice(["bf16", "fp32"])
        w = synth.Workload("s", B=B, gamma_max=G, V=V, dtype=dtype, gamma_mode="ragged",
                           temperature_mode=rnd.choice(["mixed", "scalar"]), temperature=1.0, sigma_d=synth.SIGMA_LEVELS,
                           seed=rnd.randrange(1000))
        s = synth.make_step(w, 0, DEV)
        g = torch.Generator(device=DEV).manual_seed(it)
        mask = torch.rand(B, 1, V, generator=g, device=DEV) < rnd.choice([0.0, 0.3, 0.9])
        rows = torch.rand(B, generator=g, device=DEV) < 0.5
        m = mask & rows[:, None, None]
        s["draft"] = s["draft"].masked_fill(m.expand_as(s["draft"]), float("-inf"))
        s["target"] = s["target"].masked_fill(m.expand_as(s["target"]), float("-inf"))
        am = s["draft"].float().argmax(-1).to(torch.int32)
        s["draft_tokens"] = torch.where(rows[:, None], am, s["draft_tokens"])
        T = s["temperature"].clone()
        for b in range(B):
            r = rnd.random()
            if r < 0.05:
                T[b] = 1e-6 if dtype == "fp32" else 1e-3
            elif r < 0.10:
                T[b] = 50.0
        s["temperature"] = T
        if rnd.random() < 0.5:
            s["target"][rnd.randrange(B), rnd.randrange(G + 1), rnd.randrange(V)] = float("nan")
        if rnd.random() < 0.5:
            s["draft"][rnd.randrange(B), rnd.randrange(G), rnd.randrange(V)] = float("inf")
        if rnd.random() < 0.3:
            s["draft"][rnd.randrange(B), rnd.randrange(G), :] = float("-inf")
        if rnd.random() < 0.3:
            s["uniforms"][rnd.randrange(B)] = 0.0
        gm, om = mlp_pair(synth.make_mlp(w, DEV))
        ref = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
        out = speckv.speckv_step(gpu_batch(s), s["comp"], gm)
        torch.cuda.synchronize()
        compare_step(out, ref)
        out = speckv.speckv_step(gpu_batch(s, flags=binding.SCHEDULE_SLICED | binding.READ_ALL_TARGET_ROWS), s["comp"], gm)
        torch.cuda.synchronize()
        compare_step(out, ref)
        if V >= 1000:
            out = vocab_shard.step_emulated(gpu_batch(s), rnd.choice([2, 3]), s["comp"], gm)
            torch.cuda.synchronize()
            compare_step(out, ref)
        u = torch.rand(B, G, device=DEV)
        got = speckv.speckv_sample_draft(gpu_batch(s), u)
        want = oracle.sample_draft(oracle_batch(s), u.cpu().numpy())
        np.testing.assert_array_equal(got["row_status"].cpu().numpy(), want["row_status"])
        bad = (got["tokens"].cpu().numpy() != want["tokens"]).any(1)
        assert not (bad & ((want["near"] & oracle.NEAR_CDF) == 0)).any(), (it, B, G, V, dtype)

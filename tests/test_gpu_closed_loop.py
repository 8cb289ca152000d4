"""Closed-loop controller run (gamma re-selected each step) against fixed gamma = 4 on identical streams."""
import pytest
import torch

from paper_2605_02888_b200 import closed_loop, synth

pytestmark = pytest.mark.gpu


def test_closed_loop_against_fixed_gamma_small():
    w = synth.scaled(synth.WORKLOADS["b1024_loop"], B=48, V=20000, steps=5)
    dev = torch.device("cuda", 0)
    rep = closed_loop.compare(w, w.steps, dev)
    ctl, fix = rep["controller"], rep["fixed4"]
    assert len(ctl["groups"]) == 12 and len(fix["groups"]) == 12          # 4 task clusters x 3 noise levels
    assert fix["mean_gamma_drafted"] == 4.0
    assert set(ctl["last_gamma_histogram"]) <= {2, 4, 6, 8}
    for r in (ctl, fix):
        assert 1.0 <= r["tokens_per_step"] <= w.gamma_max + 1
        assert 0.0 <= r["acceptance_rate"] <= 1.0
    assert fix["tokens_per_step"] <= 5.0                                   # at most gamma + 1 tokens per step
    # the first step is the same under both policies (gamma = 4 everywhere), and a rerun repeats itself
    again = closed_loop.run(w, w.steps, dev, "controller")
    assert again == ctl
    one_c = closed_loop.run(w, 1, dev, "controller"); one_f = closed_loop.run(w, 1, dev, "fixed")
    assert one_c["tokens_per_step"] == one_f["tokens_per_step"] and one_c["groups"] == one_f["groups"]

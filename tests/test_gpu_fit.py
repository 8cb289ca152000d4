"""Fitting the acceptance predictor on synthetic step records and driving gamma with it (Sec. 4.3-4.4)."""
import pytest
import torch

from paper_2605_02888_b200 import fit, synth

pytestmark = pytest.mark.gpu


def test_fit_and_closed_loop_small():
    w = synth.scaled(synth.WORKLOADS["b1024_loop"], B=96, V=16000)
    rep = fit.study(w, train_steps=10, eval_steps=4, device=torch.device("cuda", 0))
    assert rep["records"] == 96 * 10 and 0.0 < rep["mean_acceptance"] < 1.0
    for name in ("ridge", "mlp16"):
        assert rep["predictors"][name]["mse"] < 0.25          # better than a coin on a [0,1] target
        assert rep["predictors"][name]["corr"] > 0.0          # and it does carry signal
        assert 1.0 <= rep["policies"][name] <= w.gamma_max + 1
        assert set(int(g) for g in rep["policies"][name + "_gamma_histogram"]) <= {2, 4, 6, 8}
    assert rep["best_fixed"] in ("fixed2", "fixed4", "fixed6", "fixed8")
    assert rep["policies"]["fixed2"] <= 3.0 and rep["policies"]["fixed8"] <= 9.0

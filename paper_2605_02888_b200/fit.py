"""Fitting the acceptance predictor on records of the synthetic streams (paper Sec. 4.3-4.4).

The paper profiles speculation steps (compression level, gamma, acceptance rate and the four draft
signals per step), fits a predictor f(x, gamma) -> acceptance rate on 80 % of the records and lets
it choose gamma.  Its records are not available; this module produces the same kind of records
from the synthetic workloads by running the library with a random gamma per row and step, fits
the two cheap predictors of the paper's Table 3 in the form of Sec. 4.3 (input [Hbar, cbar, Hmax,
cmin, comp, gamma]) -- the linear (Ridge) one in closed form, the 16-hidden-unit MLP by a few
hundred Adam steps -- and compares the policies of Sec. 4.4 (fixed gamma = 4, best fixed gamma,
predictor-driven gamma) in a closed loop on later steps of the same streams.

Host-side and offline: the hot path is untouched; the fitted weights go into ``speckv.Mlp`` with
``feature_layout = 2``.

    python -m paper_2605_02888_b200.fit --workload b1024_loop --rows 256 --train-steps 24 --eval-steps 12
"""
from __future__ import annotations

import argparse
import json
from typing import Dict

import torch

from . import binding as speckv
from . import closed_loop, synth

GAMMAS = (2, 4, 6, 8)


def collect(w: synth.Workload, steps: int, device, first_step: int = 0) -> Dict[str, torch.Tensor]:
    """Step records: x = [Hbar, cbar, Hmax, cmin, comp, gamma] and the acceptance rate n / gamma of
    that step, one record per (row, step); gamma is drawn per row and step from {2,4,6,8}."""
    attrs = synth.row_attrs(w)
    mw = synth.make_mlp(w, device)
    mlp = speckv.Mlp(mw["W1"], mw["b1"], mw["W2"], mw["b2"])       # its choice is ignored here
    comp = (attrs.comp[:, 0] + 2 * attrs.comp[:, 1]).to(device)
    g = torch.Generator().manual_seed(w.seed * 31 + 7)
    choices = torch.tensor([c for c in GAMMAS if c <= w.gamma_max], dtype=torch.int32)
    xs, ys = [], []
    out = None
    for step in range(first_step, first_step + steps):
        gamma = choices[torch.randint(0, len(choices), (w.B,), generator=g)].to(device)
        s = synth.make_step(w, step, device, attrs=attrs, gamma=gamma)
        bt = speckv.Batch(draft_logits=s["draft"], target_logits=s["target"], draft_tokens=s["draft_tokens"],
                          gamma=s["gamma"], temperature=s["temperature"], uniforms=s["uniforms"])
        if out is None:
            out = speckv.StepOutputs.allocate(bt, mlp.n_out)
        res = speckv.speckv_step(bt, s["comp"], mlp, out=out)
        feat = res["feat"].clone()
        xs.append(torch.cat([feat, comp[:, None], gamma.float()[:, None]], dim=1))
        ys.append(res["n_accepted"].float() / gamma.float())
    return {"x": torch.cat(xs).cpu(), "y": torch.cat(ys).cpu()}


def fit_ridge(rec: Dict[str, torch.Tensor], lam: float = 1e-3) -> Dict[str, torch.Tensor]:
    """Closed-form ridge regression of the acceptance rate on [x, gamma] (with intercept)."""
    x = rec["x"].double()
    y = rec["y"].double()
    mu, sd = x.mean(0), x.std(0).clamp_min(1e-6)
    z = (x - mu) / sd
    A = z.T @ z + lam * len(y) * torch.eye(z.shape[1], dtype=torch.float64)
    wz = torch.linalg.solve(A, z.T @ (y - y.mean()))
    wgt = wz / sd                                               # back to raw features
    bias = y.mean() - (wgt * mu).sum()
    n_in = x.shape[1]
    return {"W1": torch.zeros(0, n_in), "b1": torch.zeros(0), "W2": wgt.float().reshape(1, n_in),
            "b2": bias.float().reshape(1)}


def fit_mlp16(rec: Dict[str, torch.Tensor], iters: int = 600, seed: int = 0) -> Dict[str, torch.Tensor]:
    """6 -> 16 ReLU -> 1 by Adam on the mean squared error; inputs are standardised for training and
    the standardisation is folded back into W1 and b1, so the library sees raw features."""
    torch.manual_seed(seed)
    x, y = rec["x"].float(), rec["y"].float()
    mu, sd = x.mean(0), x.std(0).clamp_min(1e-6)
    z = (x - mu) / sd
    W1 = (0.3 * torch.randn(16, x.shape[1])).requires_grad_()
    b1 = torch.zeros(16, requires_grad=True)
    W2 = (0.3 * torch.randn(1, 16)).requires_grad_()
    b2 = y.mean().reshape(1).clone().requires_grad_()
    opt = torch.optim.Adam([W1, b1, W2, b2], lr=2e-2)
    for _ in range(iters):
        opt.zero_grad()
        pred = torch.relu(z @ W1.T + b1) @ W2.T + b2
        loss = ((pred[:, 0] - y) ** 2).mean()
        loss.backward()
        opt.step()
    W1r = (W1 / sd).detach()
    b1r = (b1 - (W1 * (mu / sd)).sum(1)).detach()
    return {"W1": W1r.contiguous(), "b1": b1r.contiguous(), "W2": W2.detach().contiguous(), "b2": b2.detach().contiguous()}


def predict(wts: Dict[str, torch.Tensor], x: torch.Tensor) -> torch.Tensor:
    """The fitted predictor on host records (for the held-out error, not for the hot path)."""
    x = x.float()
    if wts["W1"].shape[0] == 0:
        return x @ wts["W2"][0] + wts["b2"][0]
    return (torch.relu(x @ wts["W1"].T + wts["b1"]) @ wts["W2"].T + wts["b2"])[:, 0]


def as_mlp(wts: Dict[str, torch.Tensor], device) -> "speckv.Mlp":
    t = {k: v.float().contiguous().to(device) for k, v in wts.items()}
    return speckv.Mlp(t["W1"], t["b1"], t["W2"], t["b2"], gamma_choices=GAMMAS, feature_layout=2)


def study(w: synth.Workload, train_steps: int, eval_steps: int, device) -> Dict:
    """Collect records on steps [0, train_steps), hold 20 % of them out for the prediction error, fit
    both predictors, then run the policies on steps [train_steps, train_steps + eval_steps)."""
    rec = collect(w, train_steps, device)
    n = len(rec["y"])
    perm = torch.randperm(n, generator=torch.Generator().manual_seed(1))
    tr, te = perm[: int(0.8 * n)], perm[int(0.8 * n):]
    train = {"x": rec["x"][tr], "y": rec["y"][tr]}
    report = {"workload": w.name, "rows": w.B, "records": n, "mean_acceptance": float(rec["y"].mean()), "predictors": {},
              "policies": {}}
    fitted = {"ridge": fit_ridge(train), "mlp16": fit_mlp16(train)}
    for name, wts in fitted.items():
        p = predict(wts, rec["x"][te])
        y = rec["y"][te]
        report["predictors"][name] = {"mse": float(((p - y) ** 2).mean()),
                                      "corr": float(torch.corrcoef(torch.stack([p, y]))[0, 1])}
    for gma in GAMMAS:
        if gma <= w.gamma_max:
            r = closed_loop.run(w, eval_steps, device, "fixed", gamma_fixed=gma, first_step=train_steps)
            report["policies"][f"fixed{gma}"] = r["tokens_per_step"]
    for name, wts in fitted.items():
        r = closed_loop.run(w, eval_steps, device, "controller", mlp=as_mlp(wts, device), first_step=train_steps)
        report["policies"][name] = r["tokens_per_step"]
        report["policies"][name + "_gamma_histogram"] = r["last_gamma_histogram"]
    fixed = {k: v for k, v in report["policies"].items() if k.startswith("fixed")}
    report["best_fixed"] = max(fixed, key=fixed.get)
    for name in fitted:
        report[f"{name}_vs_fixed4"] = report["policies"][name] / report["policies"]["fixed4"]
    return report


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="b1024_loop")
    ap.add_argument("--rows", type=int, default=256)
    ap.add_argument("--train-steps", type=int, default=24)
    ap.add_argument("--eval-steps", type=int, default=12)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: the library has no CPU path")
    w = synth.scaled(synth.WORKLOADS[args.workload], B=args.rows)
    print(json.dumps(study(w, args.train_steps, args.eval_steps, torch.device("cuda", 0))))


if __name__ == "__main__":
    main()

"""Closed-loop controller run on synthetic streams (the last benchmark configuration).

Every step calls the fused ``speckv_step``; under the ``controller`` policy the gamma a row uses at
step t+1 is the ``gamma_next`` the library chose for it at step t (paper Sec. 4.3: gamma is
re-selected per speculation step from the draft signals), under the ``fixed`` policy every row
keeps gamma = 4, the baseline the paper compares against (Sec. 4.4).  Both policies read the same
seeded logits, draft tokens and uniforms, because the generator produces all gamma_max positions
whatever gamma is; they differ only in how many positions they use.  Reported: tokens per step
(accepted + 1, Sec. 3.1) overall and per (task cluster, compression level) group.

This module only drives the library and keeps books; it computes none of the method.

    python -m paper_2605_02888_b200.closed_loop --workload b1024_loop --steps 20 [--rows 128]
"""
from __future__ import annotations

import argparse
import json
from typing import Dict

import torch

from . import binding as speckv
from . import synth


def run(w: synth.Workload, steps: int, device, policy: str = "controller", gamma_fixed: int = 4,
        mlp: "speckv.Mlp" = None, first_step: int = 0) -> Dict:
    """Run `steps` speculation steps of workload `w` (stream steps first_step, first_step+1, ...);
    returns tokens/step statistics and the gamma histogram of the last step.  policy: "controller"
    (gamma_next feeds the next step) or "fixed".  mlp: the controller to use (default: the
    workload's own random draw, primary 5 -> 16 -> 4 form)."""
    if policy not in ("controller", "fixed"):
        raise ValueError("policy must be 'controller' or 'fixed'")
    attrs = synth.row_attrs(w)
    if mlp is None:
        mw = synth.make_mlp(w, device)
        mlp = speckv.Mlp(mw["W1"], mw["b1"], mw["W2"], mw["b2"])
    # the paper-form predictor takes one compression scalar (0 / 1 / 2), the primary form two flags
    comp_scalar = (attrs.comp[:, 0] + 2 * attrs.comp[:, 1]).reshape(-1, 1).contiguous().to(device)
    gamma = torch.full((w.B,), min(gamma_fixed, w.gamma_max), dtype=torch.int32, device=device)
    emitted = torch.zeros(w.B, dtype=torch.int64, device=device)
    drafted = torch.zeros(w.B, dtype=torch.int64, device=device)
    out = None
    for step in range(first_step, first_step + steps):
        s = synth.make_step(w, step, device, attrs=attrs, gamma=gamma)
        comp = s["comp"] if mlp.feature_layout == 0 else comp_scalar
        bt = speckv.Batch(draft_logits=s["draft"], target_logits=s["target"], draft_tokens=s["draft_tokens"],
                          gamma=s["gamma"], temperature=s["temperature"], uniforms=s["uniforms"])
        if out is None:
            out = speckv.StepOutputs.allocate(bt, mlp.n_out)
        res = speckv.speckv_step(bt, comp, mlp, out=out)
        if int(res["row_status"].abs().sum()) != 0:
            raise RuntimeError("a row was flagged during the closed-loop run")
        emitted += res["n_accepted"].to(torch.int64) + 1
        drafted += gamma.to(torch.int64)
        if policy == "controller":
            gamma = res["gamma_next"].clone()
    tokens_per_step = emitted.double() / steps
    groups = {}
    key = attrs.cluster.to(device) * 3 + (attrs.comp[:, 0] + 2 * attrs.comp[:, 1]).to(device).long()
    for g in torch.unique(key).tolist():
        sel = key == g
        groups[f"cluster{g // 3}_level{g % 3}"] = float(tokens_per_step[sel].mean())
    return {"policy": policy, "steps": steps, "rows": w.B,
            "tokens_per_step": float(tokens_per_step.mean()),
            "acceptance_rate": float((emitted - steps).sum() / drafted.sum()),
            "mean_gamma_drafted": float(drafted.double().mean() / steps),
            "last_gamma_histogram": {int(g): int((gamma == g).sum()) for g in torch.unique(gamma).tolist()},
            "groups": groups}


def compare(w: synth.Workload, steps: int, device) -> Dict:
    """Controller policy against fixed gamma = 4 on identical streams."""
    a = run(w, steps, device, "controller")
    b = run(w, steps, device, "fixed")
    return {"workload": w.name, "controller": a, "fixed4": b,
            "tokens_per_step_ratio": a["tokens_per_step"] / b["tokens_per_step"]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="b1024_loop")
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--rows", type=int, default=None)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: the library has no CPU path")
    w = synth.WORKLOADS[args.workload]
    if args.rows:
        w = synth.scaled(w, B=args.rows)
    print(json.dumps(compare(w, args.steps, torch.device("cuda", 0))))


if __name__ == "__main__":
    main()

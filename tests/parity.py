"""Helpers shared by the GPU parity tests: feed the same seeded inputs to the CUDA path and to
the CPU oracle and compare element by element under the stated acceptance rules."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2605_02888_b200 as speckv

# Floating-point outputs: |gpu - ref| <= RTOL * |ref| + ATOL.  RTOL is the stated 1e-5 relative
# bound for fp32 accumulation; ATOL covers entropies near zero, where 1e-5 relative of a value
# like 1e-9 is below what fp32 sums of 10^5 terms can resolve.
RTOL, ATOL = 1e-5, 1e-7
# Controller scores (Eq. 1: E = a_hat * gamma + 1): a sum of terms of order one evaluated in fp32 as the task
# statement fixes; where they cancel (E near 0) what is left is the rounding of the terms, a few units of
# 2^-23 times gamma <= 8, so the absolute term is 1e-6 there.
ATOL_SCORES = 1e-6


def np_logits(t: torch.Tensor) -> np.ndarray:
    """Device logits -> host array the oracle accepts (bf16 as uint16 bit patterns)."""
    t = t.detach().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def oracle_batch(s: dict, rows=None, entropy_in_bits=False, n_threads=8, temperature_scalar=None) -> oracle.Batch:
    """oracle.Batch from a synth.make_step dict (optionally a subset of rows)."""
    if rows is not None:  # pick the rows on the device: only they cross to the host
        idx = torch.as_tensor(np.asarray(rows), dtype=torch.long)
        s = {k: (v[idx.to(v.device)] if (torch.is_tensor(v) and v.dim() >= 1 and k != "comp") else v) for k, v in s.items()}
    g = lambda k: None if s.get(k) is None else s[k].detach().cpu().numpy()
    return oracle.Batch(draft=np_logits(s["draft"]),
                        target=None if s.get("target") is None else np_logits(s["target"]),
                        draft_tokens=g("draft_tokens"), gamma=g("gamma"), temperature=g("temperature"),
                        temperature_scalar=1.0 if temperature_scalar is None else temperature_scalar,
                        uniforms=g("uniforms"), entropy_in_bits=entropy_in_bits, n_threads=n_threads)


def gpu_batch(s: dict, entropy_in_bits=False, temperature_scalar=None, flags=0) -> speckv.Batch:
    return speckv.Batch(draft_logits=s["draft"], target_logits=s.get("target"),
                        draft_tokens=s.get("draft_tokens"), gamma=s.get("gamma"),
                        temperature=s.get("temperature"),
                        temperature_scalar=1.0 if temperature_scalar is None else temperature_scalar,
                        uniforms=s.get("uniforms"), entropy_in_bits=entropy_in_bits, flags=flags)


def mlp_pair(w: dict, **kw):
    """(speckv.Mlp on the weights' device, oracle.Mlp on numpy copies)."""
    g = speckv.Mlp(w["W1"], w["b1"], w["W2"], w["b2"], **kw)
    o = oracle.Mlp(*(w[k].detach().cpu().numpy() for k in ("W1", "b1", "W2", "b2")), **kw)
    return g, o


def close(gpu, ref, what, rtol=RTOL, atol=ATOL):
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    err = np.abs(gpu - ref)
    bound = rtol * np.abs(ref) + atol
    bad = err > bound
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} outside tolerance; worst |err| "
                           f"{err[bad].max():.3e} at ref {ref[bad][err[bad].argmax()]:.6e}")
    # how many entries needed the absolute term at all
    return int((err > rtol * np.abs(ref)).sum())


def compare_step(gpu: dict, ref: dict, rows=None, check_controller=True, check_signals=True, check_verify=True,
                 mlp=None, comp=None):
    """Compare CUDA outputs (torch tensors) with oracle outputs (numpy).  Returns a report dict.
    Integer outputs must match exactly except on rows the oracle flags as near-ties.  With `mlp` (an
    oracle.Mlp) and `comp` (host array, rows already selected) the controller is also checked on its
    own: the oracle's network evaluated on the CUDA path's features must give the CUDA path's scores
    to 1e-5 relative + 1e-7, which separates the controller's arithmetic from the wobble of its inputs."""
    g = {k: (v.detach().cpu().numpy() if rows is None else v.detach().cpu().numpy()[rows]) for k, v in gpu.items()
         if v is not None}
    rep = {"rows": len(ref["row_status"])}
    np.testing.assert_array_equal(g["row_status"], ref["row_status"], err_msg="row_status")
    near = ref.get("near", np.zeros_like(ref["row_status"]))
    if check_signals:
        rep["H_abs_term"] = close(g["H"], ref["H"], "H")
        close(g["C"], ref["C"], "C")
        close(g["feat"], ref["feat"], "feat")
    if check_verify:
        n_bad = g["n_accepted"] != ref["n_accepted"]
        tok_bad = (g["out_tokens"] != ref["out_tokens"]).any(axis=1)
        rep["near_accept_rows"] = int(((near & oracle.NEAR_ACCEPT) != 0).sum())
        rep["near_cdf_rows"] = int(((near & oracle.NEAR_CDF) != 0).sum())
        # a rejection whose residual mass is below 1e-5: beyond fp32 weights; counted on its own so that a
        # workload can assert it never happens
        rep["small_residual_rows"] = int(((near & oracle.NEAR_SMALL_RESIDUAL) != 0).sum())
        # a residual draw whose threshold is within 1e-6 of a boundary in units of probability but not in units
        # of the residual's own mass: with p and q from fp32 sums, p - q is known to about 1e-7 however small
        # its total is; counted on its own
        rep["near_cdf_abs_rows"] = int(((near & oracle.NEAR_CDF_ABS) != 0).sum())
        rep["n_accepted_mismatch"] = int(n_bad.sum())
        rep["token_mismatch"] = int(tok_bad.sum())
        unflagged_n = n_bad & ((near & oracle.NEAR_ACCEPT) == 0)
        unflagged_t = tok_bad & ((near & (oracle.NEAR_ACCEPT | oracle.NEAR_CDF | oracle.NEAR_SMALL_RESIDUAL | oracle.NEAR_CDF_ABS)) == 0)
        assert not unflagged_n.any(), f"n_accepted differs on unflagged rows {np.nonzero(unflagged_n)[0][:8]}"
        assert not unflagged_t.any(), (f"out_tokens differ on unflagged rows {np.nonzero(unflagged_t)[0][:8]}: "
                                       f"gpu {g['out_tokens'][unflagged_t][:4]} ref {ref['out_tokens'][unflagged_t][:4]}")
        # structure holds on every row, flagged or not
        G1 = g["out_tokens"].shape[1]
        cols = np.arange(G1)[None, :]
        ok = g["row_status"] == 0
        assert np.all((g["n_accepted"] >= 0) & (g["n_accepted"] < G1))
        assert np.all(g["out_tokens"][ok][cols.repeat(ok.sum(), 0) > g["n_accepted"][ok][:, None]] == -1)
        assert np.all(g["out_tokens"][ok][cols.repeat(ok.sum(), 0) <= g["n_accepted"][ok][:, None]] >= 0)
    if check_controller:
        close(g["scores"], ref["scores"], "scores", atol=ATOL_SCORES)
        gm_bad = g["gamma_next"] != ref["gamma_next"]
        rep["near_gamma_rows"] = int(((near & oracle.NEAR_GAMMA) != 0).sum())
        rep["gamma_mismatch"] = int(gm_bad.sum())
        unflagged = gm_bad & ((near & oracle.NEAR_GAMMA) == 0)
        assert not unflagged.any(), f"gamma_next differs on unflagged rows {np.nonzero(unflagged)[0][:8]}"
        if mlp is not None:
            ok = g["row_status"] == 0
            own = oracle.select_gamma(g["feat"].astype(np.float64), comp, mlp)
            close(g["scores"][ok], own["scores"][ok], "scores against the oracle's network on the CUDA features",
                  rtol=1e-5, atol=1e-7)
            own_bad = (g["gamma_next"] != own["gamma_next"]) & ok & ((own["near"] & oracle.NEAR_GAMMA) == 0)
            assert not own_bad.any(), f"gamma_next is not the argmax of the CUDA path's own scores on rows {np.nonzero(own_bad)[0][:8]}"
    return rep

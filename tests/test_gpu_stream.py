"""The stream kernel (persistent CTAs, position-major order, early exit, draws from L2) against the
oracle, forced onto shapes far smaller than the ones the library hands it by default so that every
branch is met with inputs the oracle finishes in seconds: one and several slices per logit row, ragged
gamma, greedy rows, flagged rows, non-finite target rows in front of and behind the stop position."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_02888_b200 as speckv
from paper_2605_02888_b200 import binding, synth

from parity import compare_step, gpu_batch, mlp_pair, oracle_batch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
STREAM, ALL = binding.SCHEDULE_STREAM, binding.SCHEDULE_STREAM | binding.READ_ALL_TARGET_ROWS


def _both(w, step=0, flags=STREAM, edit=None):
    s = synth.make_step(w, step, DEV)
    if edit:
        edit(s)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = speckv.speckv_step(gpu_batch(s, flags=flags), s["comp"], gm)
    torch.cuda.synchronize()
    comp = s["comp"].cpu().numpy()
    ref = oracle.step(oracle_batch(s), comp, om)
    return s, out, ref, om, comp


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("V", [8, 264, 4104, 20000])
@pytest.mark.parametrize("B,G", [(1, 1), (3, 4), (37, 8), (5, 16)])
def test_stream_kernel_small_shapes(dtype, V, B, G):
    w = synth.Workload("s", B=B, gamma_max=G, V=V, dtype=dtype, gamma_mode="ragged", temperature=0.9,
                       sigma_t=1.5, sigma_d=synth.SIGMA_LEVELS, frac_identical=0.2, seed=V + B)
    for step, flags in ((0, STREAM), (1, ALL)):
        s, out, ref, om, comp = _both(w, step, flags)
        compare_step(out, ref, mlp=om, comp=comp)


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_stream_kernel_mixed_greedy_rows_and_wide_rows(dtype):
    # rows of 300,000 elements take two slices of more than 32 warp quanta each
    w = synth.Workload("s", B=24, gamma_max=6, V=300000, dtype=dtype, gamma_mode="ragged",
                       temperature_mode="mixed", sigma_d=(0.5,), frac_onehot=0.2, seed=5)
    s, out, ref, om, comp = _both(w)
    compare_step(out, ref, mlp=om, comp=comp)
    assert (s["temperature"] == 0).any() and (s["temperature"] > 0).any()


def test_stream_kernel_many_rows_repeat_bit_for_bit():
    w = synth.Workload("s", B=700, gamma_max=8, V=8192, dtype="bf16", gamma_mode="choices", temperature=0.8,
                       sigma_d=synth.SIGMA_LEVELS, frac_identical=0.1, seed=6)
    s = synth.make_step(w, 0, DEV)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    bt = gpu_batch(s, flags=STREAM)
    o = speckv.StepOutputs.allocate(bt)
    first = {k: v.clone() for k, v in speckv.speckv_step(bt, s["comp"], gm, out=o).items()}
    ref = oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om)
    compare_step(first, ref, mlp=om, comp=s["comp"].cpu().numpy())
    for _ in range(3):  # the same workspace again: which target rows are left out may differ, the results may not
        again = speckv.speckv_step(bt, s["comp"], gm, out=o)
        torch.cuda.synchronize()
        for k in first:
            assert torch.equal(first[k], again[k]), k
    full = speckv.speckv_step(gpu_batch(s, flags=ALL), s["comp"], gm)
    torch.cuda.synchronize()
    for k in first:
        assert torch.equal(first[k], full[k]), k


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_stream_kernel_flags_and_rows_behind_the_stop(dtype):
    w = synth.Workload("s", B=12, gamma_max=4, V=4096, dtype=dtype, gamma_mode="fixed", gamma_fixed=4,
                       temperature=1.0, sigma_d=(1.0,), seed=7)

    def edit(s):
        s["gamma"][0] = 0                      # bad gamma
        s["gamma"][1] = 9
        s["temperature"][2] = -1.0             # bad temperature
        s["draft_tokens"][3, 1] = w.V          # bad token
        s["draft"][4, 3, 17] = float("nan")    # non-finite draft row: flags wherever it is
        s["target"][5, 0, 100] = float("inf")  # non-finite target row at position 0: always read
        s["temperature"][6] = 0.0              # greedy row, token 0 never matches: stops at 0
        s["draft_tokens"][6, :] = 0
        s["target"][6, :, 0] = -50.0
        s["target"][6, 2, 5] = float("nan")    #   ... so a NaN at position 2 lies behind the stop
        s["uniforms"][7, 0, 0] = 0.999999      # sampled row rejected at position 0 (p/q of its token is below that)
        s["draft"][7, 0, :] = 0.0
        s["draft"][7, 0, 9] = 8.0
        s["draft_tokens"][7, 0] = 9
        s["target"][7, 0, 9] = -8.0
        s["target"][7, 3, 1] = float("nan")    #   ... a NaN behind the stop changes nothing
        s["target"][8, 4, :] = float("-inf")   # bonus row without any finite entry: flags only if reached

    for flags in (STREAM, ALL):
        s, out, ref, om, comp = _both(w, 0, flags, edit)
        st = ref["row_status"]
        assert st[0] == 1 and st[1] == 1 and st[2] == 8 and st[3] & 2 and st[4] == 4 and st[5] == 4
        assert st[6] == 0 and ref["n_accepted"][6] == 0 and st[7] == 0 and ref["n_accepted"][7] == 0
        compare_step(out, ref, mlp=om, comp=comp)


def test_stream_kernel_verify_entry_and_bits_mode():
    w = synth.Workload("s", B=9, gamma_max=5, V=12000, dtype="bf16", gamma_mode="ragged", temperature=0.7,
                       sigma_d=synth.SIGMA_LEVELS, seed=8)
    s = synth.make_step(w, 0, DEV)
    out = speckv.speckv_verify(gpu_batch(s, flags=STREAM))
    torch.cuda.synchronize()
    ref = oracle.verify(oracle_batch(s))
    compare_step(out, ref, check_controller=False, check_signals=False)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = speckv.speckv_step(gpu_batch(s, entropy_in_bits=True, flags=STREAM), s["comp"], gm)
    torch.cuda.synchronize()
    ref = oracle.step(oracle_batch(s, entropy_in_bits=True), s["comp"].cpu().numpy(), om)
    compare_step(out, ref)

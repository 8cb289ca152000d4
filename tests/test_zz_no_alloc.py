"""The allocation-free entry point, speckv_signals_static.

A serving process that has given all device memory to its framework's pool, or a plug-in that may
only touch the buffers it is handed, cannot provide the workspace speckv_signals asks for.  The
static variant carries its scratch inside the library image.  This file checks, through the C ABI,
that it returns what speckv_signals returns and what the CPU oracle computes, twice in a row on
different inputs (the second call finds the first call's leftovers in the shared array), that the
device's free memory is the same after the calls as before them, and that an over-sized batch is
refused on the host.  It is named to be collected last, so a run that stops at the first failure has already
run every other test."""
import ctypes as C

import pytest
import torch

import oracle
import paper_2605_02888_b200 as speckv
from paper_2605_02888_b200 import binding, synth

from parity import ATOL, RTOL, close, gpu_batch, oracle_batch

DEV = "cuda:0"


@pytest.mark.gpu
def test_static_scratch_matches_workspace_variant_on_two_calls_in_a_row():
    w = synth.Workload("na", B=24, gamma_max=6, V=20000, dtype="bf16", gamma_mode="ragged", temperature=0.9,
                       sigma_d=synth.SIGMA_LEVELS, seed=21)
    outs = dict(H=torch.empty(w.B, w.gamma_max, device=DEV), Cc=torch.empty(w.B, w.gamma_max, device=DEV),
                feat=torch.empty(w.B, 4, device=DEV), row_status=torch.empty(w.B, dtype=torch.int32, device=DEV))
    for step in range(2):                       # two calls in a row, different logits and gammas
        s = synth.make_step(w, step, DEV)
        if step == 1:
            s["gamma"][3] = 0                   # one flagged row: defaults and status must agree as well
        bt = gpu_batch(s)
        assert speckv.workspace_size(bt) <= binding.STATIC_SCRATCH_BYTES
        ref = {k: v.clone() for k, v in speckv.speckv_signals(bt).items()}
        want = oracle.signals(oracle_batch(s))  # the oracle's signals read the draft rows only
        for t in outs.values():
            t.fill_(-7)                         # stale contents must be overwritten
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        got = speckv.speckv_signals_static(bt, **outs)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert torch.equal(got["row_status"], ref["row_status"])
        assert (got["row_status"].cpu().numpy() == want["row_status"]).all()
        for k in ("H", "C", "feat"):
            close(got[k].cpu().numpy(), ref[k].cpu().numpy(), f"{k} against speckv_signals (call {step})", rtol=RTOL, atol=ATOL)
            close(got[k].cpu().numpy(), want[k], f"{k} against the oracle (call {step})", rtol=RTOL, atol=ATOL)


def test_static_scratch_limit_is_checked_on_the_host():
    # needs no GPU: the size check comes before any CUDA call
    L = speckv.load_library()
    b = binding._CBatch()
    b.B, b.gamma_max, b.V, b.dtype = 1024, 8, 128256, binding.BF16
    b.draft_logits = 0x1000
    b.draft_stride_b, b.draft_stride_pos = 8 * 128256, 128256
    b.temperature_scalar = 1.0
    n = C.c_size_t(0)
    assert L.speckv_workspace_size(C.byref(b), C.byref(n)) == binding.OK and n.value > binding.STATIC_SCRATCH_BYTES
    assert L.speckv_signals_static(C.byref(b), None, None, None, None, None) == binding.ERR_STATIC_LIMIT
    assert "built-in" in speckv.status_string(binding.ERR_STATIC_LIMIT)
    b.B = 0                                      # an empty batch is fine and touches nothing
    assert L.speckv_signals_static(C.byref(b), None, None, None, None, None) == binding.OK

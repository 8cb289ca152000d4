"""A bounded wait inside a kernel must end: the CTAs that draw the fresh tokens wait for their batch row's
completion flag, here nothing ever raises it, the poll limit is lowered to about a thousand polls, and the
kernel has to return with every row marked SPECKV_ROW_TIMEOUT and no token written.  Nothing hangs and
nothing faults: the wait simply runs out (about a millisecond), and the device is usable afterwards."""
import ctypes as C

import pytest
import torch

import paper_2605_02888_b200 as speckv
from paper_2605_02888_b200 import binding, synth

from parity import gpu_batch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_a_wait_that_runs_out_marks_the_rows_and_the_kernel_returns():
    L = speckv.load_library()
    B = 96
    status = torch.full((B,), 0x1234, dtype=torch.int32, device=DEV)
    tokens = torch.zeros(B, 2, dtype=torch.int32, device=DEV)
    ws = torch.empty(8 * B + 512, dtype=torch.uint8, device=DEV)
    off = (-ws.data_ptr()) % 256
    old = L.speckv_internal_set_wait_limit(1 << 10)
    try:
        with torch.cuda.device(DEV):
            rc = L.speckv_internal_wait_probe(B, status.data_ptr(), tokens.data_ptr(), ws.data_ptr() + off,
                                              ws.numel() - off, torch.cuda.current_stream().cuda_stream)
        assert rc == binding.OK
        torch.cuda.synchronize()
    finally:
        assert L.speckv_internal_set_wait_limit(old) == 1 << 10
    assert torch.all(status == binding.ROW_TIMEOUT), status[:8]
    assert torch.all(tokens == -1)
    # bad arguments come back as status codes, and the device still does ordinary work
    assert L.speckv_internal_wait_probe(0, status.data_ptr(), tokens.data_ptr(), ws.data_ptr() + off, 64, None) == binding.ERR_INVALID_ARG
    w = synth.Workload("t", B=8, gamma_max=3, V=2048, dtype="bf16", temperature=0.9, seed=1)
    s = synth.make_step(w, 0, DEV)
    out = speckv.speckv_verify(gpu_batch(s))
    torch.cuda.synchronize()
    assert torch.all(out["row_status"] == 0) and torch.all(out["n_accepted"] >= 0)

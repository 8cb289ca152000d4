"""The bounds-checked build of the library (-DSPECKV_DEBUG), which stands in for a memory checker: every
logit load and every workspace access of every kernel is compared with the extents of the call's buffers
and an access outside them is skipped and counted, never performed.  The shapes most likely to expose an
index mistake go through it here - vocabularies that are not a multiple of anything, ragged gamma, padded
and misaligned rows, broadcast rows (stride 0), the ring sweep's ragged stages, every target row read, the
sharded step, draft sampling - and the count must stay at zero with results that match the oracle.  A
self-test has the checker look at two addresses that no call registered (they are compared, not
dereferenced) to show that it would have counted them."""
import ctypes as C
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2605_02888_b200 as speckv
from paper_2605_02888_b200 import binding, build, synth, vocab_shard

from parity import compare_step, gpu_batch, mlp_pair, oracle_batch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture()
def debug_library():
    try:
        path = build.build(debug=True)
    except Exception as e:  # no compiler on this machine and no shipped binary
        if not os.path.exists(build.DEBUG_LIB_PATH):
            pytest.skip(f"bounds-checked library cannot be built here: {e}")
        path = build.DEBUG_LIB_PATH
    ordinary = speckv.load_library()
    dbg = binding.load_library(path)
    binding._lib = dbg
    rep = (C.c_ulonglong * 4)()
    assert dbg.speckv_internal_debug_report(rep, 1, 0) == binding.OK
    try:
        yield dbg
    finally:
        binding._lib = ordinary


def _violations(L, selftest=0):
    rep = (C.c_ulonglong * 4)()
    assert L.speckv_internal_debug_report(rep, 0, selftest) == binding.OK
    return list(rep)


def _check(w, flags=0, step=0):
    s = synth.make_step(w, step, DEV)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = speckv.speckv_step(gpu_batch(s, flags=flags), s["comp"], gm)
    torch.cuda.synchronize()
    compare_step(out, oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om))
    return s, gm, om


def test_no_access_leaves_its_buffers(debug_library):
    L = debug_library
    # odd vocabularies, ragged gamma, both types: sliced sweep with scalar heads and tails
    for dtype in ("fp32", "bf16"):
        for V, B, G in ((8, 1, 1), (33, 3, 4), (257, 2, 8), (4099, 3, 5), (20000, 5, 16)):
            w = synth.Workload("d", B=B, gamma_max=G, V=V, dtype=dtype, gamma_mode="ragged", temperature_mode="mixed",
                               sigma_d=synth.SIGMA_LEVELS, frac_onehot=0.2, seed=V)
            _check(w)
            _check(w, flags=binding.READ_ALL_TARGET_ROWS)
    assert _violations(L)[0] == 0, _violations(L)
    # a single batch row cut into many slices: more partials per logit row than the epilogue fetches ahead,
    # and nothing behind the row's partials but the end of the array
    for dtype, V, G in (("fp32", 32000, 8), ("bf16", 128256, 2)):
        w = synth.Workload("d", B=1, gamma_max=G, V=V, dtype=dtype, gamma_mode="fixed", gamma_fixed=G, temperature=0.5,
                           sigma_d=(0.6,), seed=50)
        _check(w)
    assert _violations(L)[0] == 0, _violations(L)
    # long rows in several slices, and enough batch rows of one slice each for the later generations of the grid
    # to find stop positions published (target rows left unread)
    for dtype, V, B in (("bf16", 300000, 6), ("fp32", 40000, 6), ("bf16", 32000, 300)):
        w = synth.Workload("d", B=B, gamma_max=3, V=V, dtype=dtype, gamma_mode="ragged", temperature=0.8,
                           sigma_d=(0.6,), seed=3)
        _check(w)
        _check(w, flags=binding.SCHEDULE_SLICED | binding.READ_ALL_TARGET_ROWS)
    assert _violations(L)[0] == 0, _violations(L)
    # the ring sweep (fp32, 384 rows and more) with rows that are not whole stages
    w = synth.Workload("d", B=400, gamma_max=2, V=4100, dtype="fp32", gamma_mode="ragged", temperature=0.9,
                       sigma_d=(0.5,), seed=4)
    _check(w)
    assert _violations(L)[0] == 0, _violations(L)
    # padded rows (stride > V), misaligned base (element-wise path), one target row broadcast to all (stride 0)
    w = synth.Workload("d", B=7, gamma_max=4, V=1000, dtype="bf16", gamma_mode="ragged", temperature=0.9,
                       sigma_d=(0.5,), seed=5)
    s = synth.make_step(w, 0, DEV)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    pad_d = torch.zeros(w.B, w.gamma_max, w.V + 24, dtype=torch.bfloat16, device=DEV)
    pad_t = torch.zeros(w.B, w.gamma_max + 1, w.V + 24, dtype=torch.bfloat16, device=DEV)
    for off in (0, 3):   # offset 3 elements: rows start 6 bytes off a 16-byte boundary
        pad_d[:, :, off:off + w.V] = s["draft"]
        pad_t[:, :, off:off + w.V] = s["target"]
        s2 = dict(s, draft=pad_d[:, :, off:off + w.V], target=pad_t[:, :, off:off + w.V])
        out = speckv.speckv_step(gpu_batch(s2), s["comp"], gm)
        torch.cuda.synchronize()
        compare_step(out, oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om))
    bro = dict(s, target=s["target"][:1].expand(w.B, -1, -1))
    out = speckv.speckv_verify(gpu_batch(bro))
    torch.cuda.synchronize()
    assert _violations(L)[0] == 0, _violations(L)
    # sharded step (ragged last shard) and draft sampling
    w = synth.Workload("d", B=9, gamma_max=5, V=4099, dtype="fp32", gamma_mode="ragged", temperature=0.8,
                       sigma_d=synth.SIGMA_LEVELS, seed=6)
    s = synth.make_step(w, 0, DEV)
    gm, om = mlp_pair(synth.make_mlp(w, DEV))
    out = vocab_shard.step_emulated(gpu_batch(s), 3, s["comp"], gm)
    torch.cuda.synchronize()
    compare_step(out, oracle.step(oracle_batch(s), s["comp"].cpu().numpy(), om))
    u = torch.rand(w.B, w.gamma_max, device=DEV)
    tok = speckv.speckv_sample_draft(gpu_batch(s), u)
    torch.cuda.synchronize()
    ref = oracle.sample_draft(oracle_batch(s), u.cpu().numpy())
    flagged = ref["near"] != 0
    assert (tok["tokens"].cpu().numpy()[~flagged] == ref["tokens"][~flagged]).all()
    assert _violations(L)[0] == 0, _violations(L)


def test_the_checker_counts_what_lies_outside(debug_library):
    L = debug_library
    before = _violations(L)[0]
    rep = _violations(L, selftest=1)
    assert rep[0] == before + 2
    if before == 0:
        assert rep[1] == 0x10 and rep[2] == 16   # the first of the two planted addresses, and its size


def test_the_ordinary_build_has_no_checker():
    rep = (C.c_ulonglong * 4)()
    assert speckv.load_library().speckv_internal_debug_report(rep, 0, 0) == binding.ERR_UNSUPPORTED

"""The debug build (libsamkv_debug.so, -DSAMKV_DEBUG_CHECKS) and the device-side checks.

A bounded wait that runs out must leave the GPU usable: the kernel records the check, drains its copies and returns;
samkv_poll_status reports it once; the next call works.  The wait is made to run out by withholding the copies of
every CTA's first tile while the spin limit is a few thousand polls (nothing faults, traps or hangs)."""
import ctypes

import pytest
import torch

from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import build, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture
def debug_library():
    path = build.build_library(debug=True)
    B.use_library(path)
    try:
        yield B.lib()
    finally:
        B.use_library(build.LIB_PATH)


def test_a_wait_that_runs_out_is_reported_and_the_next_call_works(debug_library):
    w = synth.CONFIGS["cfg1"]
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    shape = B.Shape.from_workload(w)
    _, U_tot, _ = B.samkv_layout(shape)
    h = B.Handle(shape, w.q_tokens, 64)
    ref = torch.empty((w.n_layers, w.batch, w.n_kv_heads, U_tot), dtype=torch.float32, device=DEV)
    B.samkv_score(h, shape, inp["K"], inp["Q"], w.q_tokens, inp["Qloc"], inp["Qloc"].shape[3], 1, ref)
    assert B.samkv_poll_status(h) == 0
    out = torch.full_like(ref, -5.0)
    st = debug_library.samkv_debug_score_with_lost_copy(h.h, shape.ref(), inp["K"].data_ptr(), inp["Q"].data_ptr(), w.q_tokens,
                                                        inp["Qloc"].data_ptr(), inp["Qloc"].shape[3], 1, out.data_ptr(), 4096,
                                                        ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert st == 0                                   # the call itself returns normally: the failure is on the device
    assert B.samkv_poll_status(h) == 7               # SAMKV_ERR_DEVICE_CHECK: a bounded wait ran out
    assert B.samkv_poll_status(h) == 0               # reported once
    assert bool((out == -5.0).any())                 # part of the output was never written
    out.fill_(-5.0)
    B.samkv_score(h, shape, inp["K"], inp["Q"], w.q_tokens, inp["Qloc"], inp["Qloc"].shape[3], 1, out)
    assert B.samkv_poll_status(h) == 0
    assert torch.equal(out, ref)                     # and the library works as before
    h.close()


def test_update_reports_a_token_id_outside_the_sequence():
    w = synth.ragged_workload(dtype="bf16", head_dim=128)
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    import samkv_testlib as T
    run = T.DeviceRun(w, inp).sparsify()
    R = 4
    tok = torch.tensor([[0, w.l_tot + 5, -1, 1]], dtype=torch.int32, device=DEV)
    Knew = torch.zeros((1, 1, R, w.n_kv_heads, w.head_dim), dtype=w.torch_dtype, device=DEV)
    Kc0 = run.Kc.clone()
    run.update(tok, Knew, Knew.clone(), B.SAMKV_UPDATE_OVERWRITE)
    assert run.poll() == 7                            # the bad id is skipped and reported
    # the rows of tokens 0 and 1 (protected, kept by every head) were overwritten, nothing else changed
    changed = (run.Kc.view(torch.int16) != Kc0.view(torch.int16)).any(dim=-1)
    assert int(changed.sum()) <= 2 * w.n_kv_heads
    assert run.poll() == 0

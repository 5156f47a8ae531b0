"""samkv_score_static: the scoring entry point for callers that may not allocate device memory
(a serving engine whose pool owns all of HBM; a latency-critical section where cudaMalloc's implicit
device synchronisation is unacceptable).  Its scratch is a fixed array inside the library, so it takes no
handle and no workspace.  Checked here, through the C ABI, against the regular samkv_score on two calls
in a row (the second with other inputs, so that stale scratch contents would show), plus the size limit.

The entry point keeps state inside the library (the fixed array and its cached address), so this file sorts
after the other test files and runs once they have finished.
"""
import ctypes

import pytest
import torch

from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _scores_regular(w, inp, use_bias=1):
    shape = B.Shape.from_workload(w)
    _, U_tot, _ = B.samkv_layout(shape)
    h = B.Handle(shape, w.q_tokens, 64)
    out = torch.empty((w.n_layers, w.batch, w.n_kv_heads, U_tot), dtype=torch.float32, device=DEV)
    B.samkv_score(h, shape, inp["K"], inp["Q"], w.q_tokens, inp["Qloc"], inp["Qloc"].shape[3], use_bias, out)
    torch.cuda.synchronize()
    return out


def _scores_static(w, inp, use_bias=1):
    shape = B.Shape.from_workload(w)
    _, U_tot, _ = B.samkv_layout(shape)
    out = torch.full((w.n_layers, w.batch, w.n_kv_heads, U_tot), float("nan"), dtype=torch.float32, device=DEV)
    B.samkv_score_static(shape, inp["K"], inp["Q"], w.q_tokens, inp["Qloc"], inp["Qloc"].shape[3], use_bias, out)
    torch.cuda.synchronize()
    return out


def test_static_scoring_matches_regular_entry_point_twice_in_a_row():
    # call 1: bf16, Llama head shape, 10 contexts; call 2: fp32, other shape and other values
    w1 = synth.CONFIGS["cfg1"]
    w2 = synth.ragged_workload(dtype="f32", head_dim=64, n_q_heads=6, n_kv_heads=2, block_size=4, n_init=4, n_local=8)
    in1 = {k: v.to(DEV) for k, v in synth.make_inputs(w1, "cpu").items()}
    in2 = {k: v.to(DEV) for k, v in synth.make_inputs(w2, "cpu").items()}
    ref1, ref2 = _scores_regular(w1, in1), _scores_regular(w2, in2)
    got1 = _scores_static(w1, in1)
    got2 = _scores_static(w2, in2)            # reuses the same scratch array right after call 1
    got1_again = _scores_static(w1, in1)
    for got, ref in ((got1, ref1), (got2, ref2), (got1_again, ref1)):
        assert torch.isfinite(got).all()
        # the same kernels run on both paths, so the tolerance of the score tests (1e-5 relative) is met exactly
        assert torch.allclose(got, ref, rtol=1e-5, atol=0.0)
        assert torch.equal(got, ref)
    # the bias switch is honoured on this path too
    assert torch.equal(_scores_static(w1, in1, use_bias=0), _scores_regular(w1, in1, use_bias=0))


def test_static_scoring_rejects_sizes_beyond_its_scratch_and_bad_arguments():
    w = synth.CONFIGS["cfg2"]                       # 32 layers x batch 4 x 20 contexts x 8 heads x 128 > 256 Ki floats
    shape = B.Shape.from_workload(w)
    t = torch.zeros(64, dtype=torch.float32, device=DEV)
    with pytest.raises(B.SamkvError) as e:
        B.samkv_score_static(shape, t, t, w.q_tokens, None, 1, 0, t)
    assert e.value.status == 3                      # SAMKV_ERR_WORKSPACE; nothing was launched
    one_layer = B.Shape.from_workload(w, n_layers=1)
    assert B.lib().samkv_score_static(one_layer.ref(), None, None, 1, None, 1, 0, None, None) == 1
    bad = B.Shape.from_workload(w, n_layers=1, head_dim=96)
    assert B.lib().samkv_score_static(bad.ref(), t.data_ptr(), t.data_ptr(), 1, None, 1, 0, t.data_ptr(), None) == 2
    torch.cuda.synchronize()

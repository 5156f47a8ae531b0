"""Protected-only composite cache (Sec. 3.1 "Generate generic query vector", and the no-selection ablation):
gather of the initial + local rows of every context without scores, then the prefill of the user query over it."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import samkv_oracle as O
from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import synth
from samkv_testlib import DeviceRun, check_attention

pytestmark = pytest.mark.gpu


def protected_run(w):
    inp = synth.make_inputs(w, "cuda")
    shape = B.Shape.from_workload(w)
    prot, _, _ = B.samkv_layout(shape)
    run = DeviceRun(w, inp, k_units=prot)
    return run, inp, prot


def compact_protected(run, inp):
    w = run.w
    Kc, Vc = torch.zeros_like(run.Kc), torch.zeros_like(run.Vc)
    cache_len = torch.zeros_like(run.cache_len)
    inv = torch.zeros_like(run.inv_map)
    B.samkv_compact_protected(run.handle, run.shape, inp["K"], inp["V"], Kc, Vc, run.capacity, cache_len, inv)
    torch.cuda.synchronize()
    return Kc, Vc, cache_len, inv


@pytest.mark.parametrize("name,kw", [
    ("cfg0", {}), ("cfg1", {}),
    ("cfg1", dict(block_size=64, n_init=64, n_local=128)),
    ("ragged", dict(ctx_lens=(100, 257, 64, 1000, 9), block_size=8, n_init=8, n_local=16)),
    ("ragged", dict(ctx_lens=(100, 257, 64, 1000), block_size=1, n_init=0, n_local=8)),
    ("ragged", dict(ctx_lens=(20, 5, 64), block_size=4, n_init=8, n_local=16)),          # contexts fully protected
])
def test_protected_compaction_equals_select_then_compact_and_oracle(name, kw):
    w = dataclasses.replace(synth.CONFIGS[name], **kw) if name in synth.CONFIGS else synth.ragged_workload(**kw)
    w = dataclasses.replace(w, n_layers=2, batch=2)
    run, inp, prot = protected_run(w)
    run.sparsify()                                   # scores -> select (k = protected units) -> compact
    torch.cuda.synchronize()
    Kc, Vc, cache_len, inv = compact_protected(run, inp)
    assert torch.equal(Kc.view(torch.uint8), run.Kc.view(torch.uint8))
    assert torch.equal(Vc.view(torch.uint8), run.Vc.view(torch.uint8))
    assert torch.equal(inv, run.inv_map) and torch.equal(cache_len, run.cache_len)
    # the oracle's gather of the protected units
    nb, off = O.unit_layout(w.ctx_offsets, w.block_size)
    units = [off[c] + m for c in range(w.n_ctx)
             for m in O.protected_units(w.ctx_lens[c], w.block_size, w.n_init, w.n_local)]
    toks = O.units_to_tokens(np.asarray(units), w.ctx_offsets, w.block_size)
    assert int(cache_len[1, 1]) == len(toks) == run.S
    idx = torch.from_numpy(toks)
    for h in range(w.n_kv_heads):
        assert torch.equal(Kc[1, 1, h, :run.S].cpu().view(torch.uint8), inp["K"][1, 1, h].cpu()[idx].view(torch.uint8))
        assert torch.equal(Vc[1, 1, h, :run.S].cpu().view(torch.uint8), inp["V"][1, 1, h].cpu()[idx].view(torch.uint8))
    assert run.poll() == 0


def test_generic_query_prefill_over_the_composite_cache():
    """The user query chunk attends over the protected rows of all contexts plus its own causal prefix."""
    w = synth.CONFIGS["cfg1"]
    run, inp, prot = protected_run(w)
    Kc, Vc, cache_len, inv = compact_protected(run, inp)
    run.Kc, run.Vc, run.cache_len = Kc, Vc, cache_len
    Kc_before, Vc_before = Kc[0, 0].clone(), Vc[0, 0].clone()
    Og, lse = run.attn(0, inp["Qa"][0], inp["Kq"][0], inp["Vq"][0])
    torch.cuda.synchronize()
    assert run.poll() == 0 and int(cache_len[0, 0]) == run.S + w.q_tokens
    check_attention(w, Kc_before, Vc_before, run.S, inp["Qa"][0, 0], inp["Kq"][0, 0], inp["Vq"][0, 0], Og[0], lse[0])


def test_no_selection_ablation_is_a_subset_of_the_selected_cache():
    """Every row of the protected-only cache also sits in the cache built with a budget, in the same order."""
    w = synth.CONFIGS["cfg1"]
    inp = synth.make_inputs(w, "cuda")
    full = DeviceRun(w, inp).sparsify()
    run, _, prot = protected_run(w)
    Kc, Vc, cache_len, inv = compact_protected(run, inp)
    torch.cuda.synchronize()
    inv_p, inv_f = inv[0, 0, 0].cpu().numpy(), full.inv_map[0, 0, 0].cpu().numpy()
    kept_p = np.nonzero(inv_p >= 0)[0]
    assert (inv_f[kept_p] >= 0).all() and np.all(np.diff(inv_f[kept_p]) > 0)
    assert torch.equal(Kc[0, 0, 0, :run.S].cpu(), full.Kc[0, 0, 0].cpu()[torch.from_numpy(inv_f[kept_p]).long()])

"""GPU parity of the cross-layer alignment plan (Sec. 3.3): flags, merged axis and per-layer forward lists
must equal the oracle's exactly (integer work, bit-exact)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import samkv_oracle as O
from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import synth
from samkv_testlib import DeviceRun

pytestmark = pytest.mark.gpu


def run_align(run, inv_map, tok_ids, run_capacity):
    w = run.w
    dev = inv_map.device
    L, Bt = w.n_layers, w.batch
    flags = torch.full((L, Bt, w.l_tot), 0xAA, dtype=torch.uint8, device=dev)
    merged = torch.full((Bt, w.l_tot), -9, dtype=torch.int32, device=dev)
    merged_len = torch.full((Bt,), -9, dtype=torch.int32, device=dev)
    run_ids = torch.full((L, Bt, run_capacity), -9, dtype=torch.int32, device=dev)
    run_len = torch.full((L, Bt), -9, dtype=torch.int32, device=dev)
    B.samkv_align(run.handle, run.shape, inv_map, tok_ids, flags, merged, merged_len, run_ids, run_len)
    torch.cuda.synchronize()
    return flags.cpu().numpy(), merged.cpu().numpy(), merged_len.cpu().numpy(), run_ids.cpu().numpy(), run_len.cpu().numpy()


def check_against_oracle(w, inv_map, tok_ids, out, batches=None):
    flags, merged, merged_len, run_ids, run_len = out
    inv = inv_map.cpu().numpy()
    tok = np.full((w.n_layers, 1), -1) if tok_ids is None else tok_ids.cpu().numpy()
    for b in (range(w.batch) if batches is None else batches):
        f_or, m_or, r_or = O.align_layers(inv[:, b], tok)
        assert np.array_equal(flags[:, b], f_or), f"flags b{b}"
        assert merged_len[b] == len(m_or)
        assert np.array_equal(merged[b, :len(m_or)], m_or) and (merged[b, len(m_or):] == -1).all()
        for n in range(w.n_layers):
            assert run_len[n, b] == len(r_or[n]), f"run_len l{n} b{b}"
            assert np.array_equal(run_ids[n, b, :len(r_or[n])], r_or[n]), f"run_ids l{n} b{b}"
            assert (run_ids[n, b, len(r_or[n]):] == -1).all()


def random_inv_map(L, Bt, Hkv, L_tot, p, seed, device="cuda"):
    g = torch.Generator(device="cpu").manual_seed(seed)
    kept = torch.rand((L, Bt, Hkv, L_tot), generator=g) < p
    return torch.where(kept, torch.cumsum(kept.int(), dim=-1) - 1, torch.full_like(kept, -1, dtype=torch.int32)).to(
        torch.int32).to(device)


def small_run(L=4, Bt=2, ctx_lens=(300, 257, 130), seed=7):
    w = dataclasses.replace(synth.ragged_workload(ctx_lens=ctx_lens, seed=seed), n_layers=L, batch=Bt)
    inp = synth.make_inputs(w, "cuda")
    return w, DeviceRun(w, inp)


def test_align_after_fixed_budget_selection():
    """Real selection output: layers and heads keep different middle tokens; recompute lists drawn per layer."""
    w, run = small_run()
    run.sparsify()
    torch.cuda.synchronize()
    g = torch.Generator().manual_seed(3)
    tok = torch.stack([torch.randperm(w.l_tot, generator=g)[:40] for _ in range(w.n_layers)]).to(torch.int32)
    tok[:, ::7] = -1
    # make sure kept tokens are listed too (random ids are mostly blanks at a 15 % budget)
    inv0 = run.inv_map[:, 0, 0].cpu()
    for n in range(w.n_layers):
        kept = torch.nonzero(inv0[n] >= 0).flatten()
        tok[n, 1:21:2] = kept[torch.randperm(len(kept), generator=g)[:10]].to(torch.int32)
    tok = tok.cuda()
    out = run_align(run, run.inv_map, tok, run_capacity=w.n_layers * 40)
    check_against_oracle(w, run.inv_map, tok, out)
    assert out[4].max() > 0 and run.poll() == 0


@pytest.mark.parametrize("L,Bt,Hkv,p,seed", [(1, 1, 1, 0.5, 0), (6, 2, 2, 0.3, 1), (3, 1, 8, 0.05, 2), (5, 3, 2, 0.0, 3),
                                             (2, 1, 2, 1.0, 4)])
def test_align_random_maps(L, Bt, Hkv, p, seed):
    w = dataclasses.replace(synth.ragged_workload(ctx_lens=(211, 190), n_q_heads=Hkv * 2, n_kv_heads=Hkv, seed=seed),
                            n_layers=L, batch=Bt)
    run = DeviceRun(w, synth.make_inputs(w, "cuda"))
    inv = random_inv_map(L, Bt, Hkv, w.l_tot, p, seed)
    g = torch.Generator().manual_seed(seed)
    tok = torch.stack([torch.randperm(w.l_tot, generator=g)[:25] for _ in range(L)]).to(torch.int32).cuda()
    out = run_align(run, inv, tok, run_capacity=w.l_tot)
    check_against_oracle(w, inv, tok, out)
    assert run.poll() == 0


def test_align_without_recompute_lists():
    w, run = small_run(L=3, Bt=1)
    inv = random_inv_map(3, 1, w.n_kv_heads, w.l_tot, 0.2, 11)
    out = run_align(run, inv, None, run_capacity=4)
    check_against_oracle(w, inv, None, out)
    assert (out[4] == 0).all() and (out[0] <= 1).all()


def test_align_list_capacity_and_bad_ids_are_reported():
    w, run = small_run(L=3, Bt=1)
    inv = random_inv_map(3, 1, w.n_kv_heads, w.l_tot, 1.0, 12)
    tok = torch.arange(30, dtype=torch.int32).repeat(3, 1).cuda()
    flags, merged, merged_len, run_ids, run_len = run_align(run, inv, tok, run_capacity=8)
    assert run_len.flatten().tolist() == [30, 30, 30]            # the full counts
    assert np.array_equal(run_ids[0, 0], np.arange(8))            # truncated, still ascending
    assert run.poll() != 0                                        # and recorded
    assert run.poll() == 0
    tok[1, 3] = w.l_tot                                           # one past the last token
    run_align(run, inv, tok, run_capacity=64)
    assert run.poll() != 0


def test_align_bench_shape_sample():
    """cfg2's token axis (30 720 tokens, 8 heads) on 4 layers; the oracle checks one batch element."""
    w = dataclasses.replace(synth.CONFIGS["cfg2"], name="align_cfg2", n_layers=4, batch=2)
    inp = synth.make_inputs(w, "cuda")
    run = DeviceRun(w, inp).sparsify()
    torch.cuda.synchronize()
    sel_tok = torch.stack([torch.nonzero(run.inv_map[n, 0, 0] >= 0).flatten() for n in range(w.n_layers)])
    tok, _, _ = synth.make_recompute(w, inp["K"], inp["V"], sel_tok[:, None, :], 690)
    out = run_align(run, run.inv_map, tok, run_capacity=4 * 690)
    flags, merged, merged_len, run_ids, run_len = out
    assert run.poll() == 0
    # properties at full width: nesting of the forward lists and list/flag agreement
    for b in range(w.batch):
        for n in range(w.n_layers):
            ids = run_ids[n, b, :run_len[n, b]]
            assert np.all(np.diff(ids) > 0)
            assert np.array_equal(ids, np.nonzero(flags[n, b] & 6)[0])
            if n + 1 < w.n_layers:
                assert np.array_equal(np.nonzero(flags[n, b] & 4)[0], run_ids[n + 1, b, :run_len[n + 1, b]])
        assert np.array_equal(merged[b, :merged_len[b]], np.nonzero((flags[:, b] & 1).any(axis=0))[0])
    # the oracle on a 2 048-token window of batch element 1 (its loops are O(L * L_tot * R))
    lo, hi = 1536 * 3 - 700, 1536 * 3 + 1348
    inv_win = run.inv_map[:, 1:2, :, lo:hi].cpu().numpy()[:, 0]
    tok_np = tok.cpu().numpy()
    tok_win = np.where((tok_np >= lo) & (tok_np < hi), tok_np - lo, -1)
    f_or, m_or, r_or = O.align_layers(inv_win, tok_win)
    assert np.array_equal(flags[:, 1, lo:hi], f_or)

"""GPU-vs-oracle parity, stage by stage, through the C ABI (libsamkv.so via the ctypes binding).

Acceptance (stated in samkv_testlib): selected index sets exact except inside the 1e-5 relative
tie band around the oracle's k-th score; compaction bit-exact; overwrite bit-exact; fusion within
one bf16 ulp (bf16) / 1e-5 relative (fp32); attention max-abs <= 2e-2 (bf16) / 1e-4 (fp32).
"""
import numpy as np
import pytest
import torch

from oracle import samkv_oracle as O
from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import synth
from samkv_testlib import (DeviceRun, check_attention, check_compact, check_scores, check_selection, check_update,
                           oracle_k_units, oracle_scores, to_f64)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def full_check(w, inp=None, k_units=None, use_bias=True, with_qloc=True, append=True, layers=None, batches=None):
    """Sparsify + prefill attention for a workload; every stage against the oracle."""
    inp = inp if inp is not None else {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp, k_units=k_units, use_bias=use_bias, with_qloc=with_qloc).sparsify()
    if k_units is None:
        assert run.k_units == oracle_k_units(w)
    torch.cuda.synchronize()
    sel = run.sel.cpu().numpy()
    n_diff = 0
    ls = list(layers if layers is not None else range(w.n_layers))
    bs = list(batches if batches is not None else range(w.batch))
    for l in ls:
        for b in bs:
            q, s, u = oracle_scores(w, inp, l, b, use_bias, with_qloc)
            check_scores(w, run, l, b, q, u)
            n_diff += check_selection(w, run.k_units, sel[l, b], u, where=f"{w.name} l{l} b{b}")
            check_compact(w, run, l, b, sel[l, b])
    for l in ls:
        Kc_before, Vc_before = run.Kc[l].clone(), run.Vc[l].clone()
        Kq = inp["Kq"][l] if append else None
        Vq = inp["Vq"][l] if append else None
        Og, lse = run.attn(l, inp["Qa"][l], Kq, Vq)
        torch.cuda.synchronize()
        for b in bs:
            err, K2, V2, n = check_attention(w, Kc_before[b], Vc_before[b], run.S, inp["Qa"][l, b],
                                             Kq[b] if append else None, Vq[b] if append else None, Og[b], lse[b])
            assert int(run.cache_len[l, b]) == n
            if append:    # appended rows are in the cache, bit-exact, right after the kept tokens
                assert np.array_equal(to_f64(run.Kc[l, b][:, run.S:n]), K2[:, run.S:n])
                assert np.array_equal(to_f64(run.Vc[l, b][:, run.S:n]), V2[:, run.S:n])
    assert run.poll() == 0
    return run, n_diff


def test_cfg0_tiny_fp32():
    run, _ = full_check(synth.CONFIGS["cfg0"])
    assert run.S == 152


def test_cfg1_llama_shape_bf16():
    run, _ = full_check(synth.CONFIGS["cfg1"])
    assert run.S == 1530


@pytest.mark.parametrize("dtype,hd", [("f32", 64), ("f32", 128), ("bf16", 64), ("bf16", 128)])
def test_ragged_contexts_token_mode(dtype, hd):
    w = synth.ragged_workload(dtype=dtype, head_dim=hd, n_q_heads=6, n_kv_heads=2, q_tokens=5)
    full_check(w)


@pytest.mark.parametrize("B_,ni,nl", [(16, 16, 32), (64, 64, 128), (4, 4, 8), (2, 0, 2)])
def test_block_mode_ragged(B_, ni, nl):
    w = synth.ragged_workload(ctx_lens=(300, 1027, 256, 2000), dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=2,
                              q_tokens=9, block_size=B_, n_init=ni, n_local=nl, budget_bp=2000)
    full_check(w)


def test_block_mode_cfg1_paper_blocks():
    full_check(synth.CONFIGS["cfg1"].replace(name="cfg1_b64", block_size=64, n_init=64, n_local=128, budget_bp=3000))
    full_check(synth.CONFIGS["cfg0"].replace(name="cfg0_b16", block_size=16, n_init=16, n_local=32, budget_bp=4000))


def test_single_context_and_bias_switches():
    w = synth.ragged_workload(ctx_lens=(700,), dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=4, q_tokens=3)
    run, _ = full_check(w)                                        # D = 1: Q^ = Q_que
    w4 = synth.ragged_workload(dtype="f32", head_dim=64)
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w4, "cpu").items()}
    a, _ = full_check(w4, inp, use_bias=False)
    b, _ = full_check(w4, inp, with_qloc=False)
    assert torch.equal(a.scores, b.scores) and torch.equal(a.sel, b.sel)
    c, _ = full_check(w4, inp, use_bias=True)
    assert not torch.equal(a.scores, c.scores)


def test_budget_edges_protected_only_and_full():
    w = synth.ragged_workload(dtype="bf16", head_dim=128, n_q_heads=4, n_kv_heads=2)
    shape = B.Shape.from_workload(w)
    prot, _, _ = B.samkv_layout(shape)
    run, _ = full_check(w, k_units=prot)                          # the "no selection" ablation: protected only
    assert run.S == sum(prot)
    nb = list(w.ctx_lens)
    run, _ = full_check(w, k_units=nb, append=False)              # 100 %
    assert run.S == w.l_tot
    # 100 % budget, no update: identical to full attention over the concatenated contexts
    inp = run.inp
    assert torch.equal(run.Kc[0, 0][:, :w.l_tot], inp["K"][0, 0]) and torch.equal(run.Vc[0, 0][:, :w.l_tot], inp["V"][0, 0])
    Og, _ = run.attn(0, inp["Qa"][0])
    out, *_ = O.attention(to_f64(inp["K"][0, 0]), to_f64(inp["V"][0, 0]), w.l_tot, to_f64(inp["Qa"][0, 0]))
    assert np.abs(to_f64(Og[0]) - out).max() <= 2e-2


def test_ties_lower_index_wins():
    """Duplicated key rows give exactly equal scores on both sides; the lower index must be kept."""
    w = synth.ragged_workload(ctx_lens=(400, 600), dtype="bf16", head_dim=128, n_q_heads=4, n_kv_heads=2, n_init=4,
                              n_local=4, budget_bp=1000)
    inp = synth.make_inputs(w, "cpu")
    K = inp["K"]
    g = torch.Generator().manual_seed(5)
    for h in range(2):
        for c, (lo, hi) in enumerate(((0, 400), (400, 1000))):
            src = torch.randint(lo + 10, hi - 10, (60,), generator=g)
            dst = torch.randint(lo + 10, hi - 10, (60,), generator=g)
            K[0, 0, h, dst] = K[0, 0, h, src]
    # and a context where every middle key is the same row: the kept middle units must be the first ones
    K[0, 0, 0, 404:996] = K[0, 0, 0, 500]
    inp = {k: v.to(DEV) for k, v in inp.items()}
    run, n_diff = full_check(w, inp)
    sel = run.sel[0, 0, 0].cpu().numpy()
    k0, k1 = run.k_units
    mid = sel[k0 + 4: k0 + k1 - 4]
    assert list(mid) == list(range(404, 404 + len(mid)))


@pytest.mark.parametrize("mode", [B.SAMKV_UPDATE_OVERWRITE, B.SAMKV_UPDATE_FUSION])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_update_overwrite_and_fusion(mode, dtype):
    """Reduced cfg2: outlier channels, sink keys, 15 % of the kept tokens recomputed, then attention."""
    w = synth.CONFIGS["cfg2"].replace(name="cfg2_small", n_layers=2, batch=2, ctx_lens=(384, 256, 512), dtype=dtype,
                                      q_tokens=16)
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp).sparsify()
    sel = run.sel.cpu().numpy()
    toks0 = np.stack([[O.units_to_tokens(sel[l, b, 0], w.ctx_offsets, 1) for b in range(w.batch)]
                      for l in range(w.n_layers)])
    R = (w.recompute_share_bp * run.S) // 10000
    tok_ids, Knew, Vnew = synth.make_recompute(w, inp["K"], inp["V"], torch.from_numpy(toks0), R)
    tok_ids[0, 3] = -1                                             # a skipped entry
    Kc0, Vc0 = run.Kc.clone(), run.Vc.clone()
    run.update(tok_ids, Knew, Vnew, mode)
    torch.cuda.synchronize()
    inv = run.inv_map.cpu().numpy()
    n_blank = 0
    for l in range(w.n_layers):
        for b in range(w.batch):
            check_update(w, Kc0[l, b], Vc0[l, b], run.Kc[l, b], run.Vc[l, b], inv[l, b], tok_ids[l].cpu().numpy(),
                         Knew[l, b], Vnew[l, b], mode)
            n_blank += int((inv[l, b][1:, tok_ids[l].cpu().numpy().clip(0)] < 0).sum())
        Og, lse = run.attn(l, inp["Qa"][l], inp["Kq"][l], inp["Vq"][l])
        for b in range(w.batch):
            check_attention(w, run.Kc[l, b].clone(), run.Vc[l, b].clone(), run.S, inp["Qa"][l, b], inp["Kq"][l, b],
                            inp["Vq"][l, b], Og[b], lse[b])
    assert n_blank > 0          # some heads did not keep some recomputed tokens: the skip rule was exercised
    assert run.poll() == 0


def test_decode_steps_append_to_compact_cache():
    """Reduced cfg3: sparsify, prefill a 32-token chunk, then decode steps of one token each."""
    w = synth.CONFIGS["cfg3"].replace(name="cfg3_small", batch=3, ctx_lens=(512, 768, 300), decode_steps=12)
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp).sparsify()
    Og, lse = run.attn(0, inp["Qa"][0], inp["Kq"][0], inp["Vq"][0])
    Kc_ref = [to_f64(run.Kc[0, b]) for b in range(w.batch)]
    Vc_ref = [to_f64(run.Vc[0, b]) for b in range(w.batch)]
    n = run.S + w.q_tokens
    g = torch.Generator().manual_seed(9)
    for step in range(w.decode_steps):
        q = torch.randn((w.batch, 1, w.n_q_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        kq = torch.randn((w.batch, 1, w.n_kv_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        vq = torch.randn((w.batch, 1, w.n_kv_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        Os, ls = run.attn(0, q, kq, vq)
        for b in range(w.batch):
            out, l2, Kc_ref[b], Vc_ref[b], n2 = O.attention(Kc_ref[b], Vc_ref[b], n, to_f64(q[b]), to_f64(kq[b]), to_f64(vq[b]))
            assert np.abs(to_f64(Os[b]) - out).max() <= 2e-2
            assert np.abs(to_f64(ls[b]) - l2).max() <= 2e-2
        n += 1
        assert run.cache_len.cpu().tolist() == [[n] * w.batch]
    for b in range(w.batch):
        assert np.array_equal(to_f64(run.Kc[0, b])[:, :n], Kc_ref[b][:, :n])
    assert run.poll() == 0


@pytest.mark.parametrize("T_q,G", [(1, 4), (8, 4), (3, 8), (40, 4), (64, 8)])
def test_attention_row_tilings_and_long_cache(T_q, G):
    """Every row tiling of the bf16 kernel (16 / 64 / 128 packed rows per CTA), with many KV splits."""
    w = synth.ragged_workload(ctx_lens=(3000, 2500), dtype="bf16", head_dim=128, n_q_heads=2 * G, n_kv_heads=2,
                              q_tokens=T_q, n_init=16, n_local=32, budget_bp=9000)
    full_check(w)


def test_results_are_deterministic():
    w = synth.CONFIGS["cfg1"]
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    outs = []
    for _ in range(3):
        run = DeviceRun(w, inp).sparsify()
        Og, lse = run.attn(0, inp["Qa"][0], inp["Kq"][0], inp["Vq"][0])
        outs.append((run.scores.clone(), run.sel.clone(), run.Kc.clone(), Og.clone(), lse.clone()))
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))


def test_error_codes_launch_nothing():
    w = synth.CONFIGS["cfg0"]
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp).sparsify()
    torch.cuda.synchronize()
    sel_before = run.sel.clone()
    with pytest.raises(B.SamkvError) as e:
        B.samkv_select(run.handle, run.shape, run.scores, [5, 38, 38, 38], run.sel)         # below the protected count
    assert e.value.status == 5
    with pytest.raises(B.SamkvError) as e:
        B.samkv_select(run.handle, run.shape, run.scores, [257, 38, 38, 38], run.sel)
    assert e.value.status == 5
    with pytest.raises(B.SamkvError) as e:
        B.samkv_compact(run.handle, run.shape, inp["K"], inp["V"], run.sel, run.k_units, run.Kc, run.Vc, 100,
                        run.cache_len, None)
    assert e.value.status == 4
    with pytest.raises(B.SamkvError) as e:                                                   # misaligned K
        B.samkv_score(run.handle, run.shape, inp["K"].view(-1)[1:], inp["Q"], 16, None, 1, 0, run.scores, None)
    assert e.value.status == 1
    bad = B.Shape(1, 1, 4, 2, 96, w.ctx_offsets, 1, 4, 8, "f32")
    with pytest.raises(B.SamkvError) as e:
        B.samkv_score(run.handle, bad, inp["K"], inp["Q"], 16, None, 1, 0, run.scores, None)
    assert e.value.status == 2
    with pytest.raises(B.SamkvError) as e:                                                   # Kq without Vq
        B.samkv_attn(run.handle, run.shape, 0, run.Kc, run.Vc, run.capacity, run.cache_len, inp["Qa"][0], 16,
                     inp["Kq"][0], None, 0.0, torch.empty_like(inp["Qa"][0]))
    assert e.value.status == 1
    torch.cuda.synchronize()
    assert torch.equal(run.sel, sel_before) and run.poll() == 0


def test_append_past_capacity_is_reported_not_fatal():
    """A full cache: the append is skipped, a device check is recorded, the context stays usable."""
    w = synth.CONFIGS["cfg0"]
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp, extra_capacity=8).sparsify()               # room for 8 tokens, chunk has 16
    Og, _ = run.attn(0, inp["Qa"][0], inp["Kq"][0], inp["Vq"][0])
    assert run.poll() == 7
    assert int(run.cache_len[0, 0]) == run.S
    assert run.poll() == 0                                          # cleared by the previous poll
    Og2, _ = run.attn(0, inp["Qa"][0])                              # cache-only attention still works
    check_attention(w, run.Kc[0, 0], run.Vc[0, 0], run.S, inp["Qa"][0, 0], None, None, Og2[0])
    assert torch.equal(Og, Og2)


def test_compact_gathers_rows_from_pinned_host_memory():
    """V (and K) may stay in pinned host memory; only the kept rows cross the bus.  Same bits as from the device."""
    w = synth.CONFIGS["cfg1"]
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp).sparsify()
    torch.cuda.synchronize()
    Kc_dev, Vc_dev = run.Kc.clone(), run.Vc.clone()
    V_host = inp["V"].cpu().pin_memory()
    run.Kc.zero_(); run.Vc.zero_()
    B.samkv_compact(run.handle, run.shape, inp["K"], V_host, run.sel, run.k_units, run.Kc, run.Vc, run.capacity,
                    run.cache_len, run.inv_map)
    torch.cuda.synchronize()
    assert torch.equal(run.Kc, Kc_dev) and torch.equal(run.Vc, Vc_dev)
    check_compact(w, run, 0, 0, run.sel[0, 0].cpu().numpy())
    # K too (the deployment with block representatives resident: neither K nor V is uploaded as a whole)
    K_host = inp["K"].cpu().pin_memory()
    run.Kc.zero_(); run.Vc.zero_()
    B.samkv_compact(run.handle, run.shape, K_host, V_host, run.sel, run.k_units, run.Kc, run.Vc, run.capacity,
                    run.cache_len, run.inv_map)
    torch.cuda.synchronize()
    assert torch.equal(run.Kc, Kc_dev) and torch.equal(run.Vc, Vc_dev)
    with pytest.raises(ValueError):                                   # pageable host memory is refused by the binding
        B.samkv_compact(run.handle, run.shape, inp["K"], inp["V"].cpu(), run.sel, run.k_units, run.Kc, run.Vc,
                        run.capacity, run.cache_len, run.inv_map)
    assert run.poll() == 0


def test_many_contexts_and_raw_local_query_rows():
    """128 contexts (the library's maximum), ragged lengths, raw local Q rows (T_loc = n_local) in bf16, G = 8."""
    g = torch.Generator().manual_seed(3)
    lens = tuple(int(x) for x in torch.randint(40, 90, (128,), generator=g))
    w = synth.Workload("many_ctx", 1, 2, 16, 2, 128, "bf16", lens, 4, budget_bp=2500, block_size=1, n_init=4, n_local=8,
                       t_loc=8, rope_base=10000.0, seed=31)
    full_check(w)
    shape = B.Shape.from_workload(w.replace(ctx_lens=lens + (50,)))
    with pytest.raises(B.SamkvError) as e:                              # 129 contexts: refused, not truncated
        B.samkv_budget_units(shape, 1500)
    assert e.value.status == 2


@pytest.mark.parametrize("dtype,hd,lo,hi,n", [("bf16", 128, 24, 25, 20), ("f32", 64, 16, 41, 30), ("f32", 128, 3, 11, 40),
                                              ("bf16", 64, 33, 71, 25), ("bf16", 128, 100, 400, 7)])
def test_short_contexts_share_scoring_tiles(dtype, hd, lo, hi, n):
    """Contexts much shorter than a 32 KB scoring tile: a tile then spans several contexts and every row is scored
    with the personalised query of its own context (Eq. 1).  The third case has more contexts per tile than the
    kernel carries queries for (it falls back to one tile per context), the last one mixes both regimes."""
    g = torch.Generator().manual_seed(hd + n)
    lens = tuple(int(x) for x in torch.randint(lo, hi, (n,), generator=g))
    w = synth.Workload("short_ctx", 2, 2, 8, 2, hd, dtype, lens, 6, budget_bp=3000, block_size=1, n_init=1, n_local=2,
                       t_loc=2, rope_base=10000.0, seed=5)
    full_check(w)


def test_large_context_uses_block_wide_select_and_head_dim_64_prefill():
    """One context of 20 000 tokens (block-wide radix select, several passes over shared memory) next to a short
    one; head_dim 64 with 160 packed rows goes through the 64-row mma.sync tiling."""
    w = synth.Workload("big_ctx", 1, 1, 8, 2, 64, "bf16", (20000, 300), 20, budget_bp=1000, block_size=1, n_init=16,
                       n_local=32, t_loc=1, rope_base=10000.0, seed=41)
    run, _ = full_check(w)
    assert run.S == 2000 + 48


def test_paper_block_settings_on_decode_shape():
    """Block size 64 with 1 initial and 2 local blocks (the paper's settings) on a reduced cfg3: block-mean scores,
    block selection, then prefill chunk and a few decode steps."""
    w = synth.CONFIGS["cfg3"].replace(name="cfg3_b64", batch=2, ctx_lens=(2048, 1999, 1024), block_size=64, n_init=64,
                                      n_local=128, budget_bp=2500, decode_steps=3)
    run, _ = full_check(w)
    inp = run.inp
    g = torch.Generator().manual_seed(19)
    n = run.S + w.q_tokens
    ref = [(to_f64(run.Kc[0, b]), to_f64(run.Vc[0, b])) for b in range(w.batch)]
    for step in range(w.decode_steps):
        q = torch.randn((w.batch, 1, w.n_q_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        kq = torch.randn((w.batch, 1, w.n_kv_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        vq = torch.randn((w.batch, 1, w.n_kv_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        Os, _ = run.attn(0, q, kq, vq)
        for b in range(w.batch):
            out, _, K2, V2, _ = O.attention(ref[b][0], ref[b][1], n, to_f64(q[b]), to_f64(kq[b]), to_f64(vq[b]))
            ref[b] = (K2, V2)
            assert np.abs(to_f64(Os[b]) - out).max() <= 2e-2
        n += 1
    assert run.poll() == 0


def test_context_beyond_shared_memory_is_refused():
    w = synth.Workload("huge_ctx", 1, 1, 4, 2, 64, "f32", (60000,), 2, n_init=4, n_local=8, t_loc=1, seed=5)
    shape = B.Shape.from_workload(w)
    with pytest.raises(B.SamkvError) as e:
        B.samkv_budget_units(shape, 1500)                               # more units in one context than the select kernel holds
    assert e.value.status == 2


def test_chunked_prefill_on_the_tensor_memory_kernel():
    """Three consecutive 64-token chunks on the same layer (256 packed rows per KV head, so every call takes the
    tcgen05 kernel and its dependent-launch chain: append -> attention -> merge).  Each call must see the cache
    length and the rows the previous call left, then a cache-only call must see all three chunks."""
    w = synth.CONFIGS["cfg1"].replace(name="cfg1_chunks", batch=2, q_tokens=64, ctx_lens=(1024, 700, 1300))
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp, extra_capacity=3 * 64).sparsify()
    torch.cuda.synchronize()
    Kc_ref = [to_f64(run.Kc[0, b]) for b in range(w.batch)]
    Vc_ref = [to_f64(run.Vc[0, b]) for b in range(w.batch)]
    n = run.S
    g = torch.Generator().manual_seed(17)
    outs = []
    for chunk in range(3):                                      # launched back to back, no host synchronisation
        q = torch.randn((w.batch, 64, w.n_q_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        kq = torch.randn((w.batch, 64, w.n_kv_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        vq = torch.randn((w.batch, 64, w.n_kv_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
        outs.append((q, kq, vq) + run.attn(0, q, kq, vq))
    q_last = torch.randn((w.batch, 64, w.n_q_heads, w.head_dim), generator=g).to(w.torch_dtype).to(DEV)
    O_last, lse_last = run.attn(0, q_last)                      # cache only, right behind an appending call
    torch.cuda.synchronize()
    assert run.poll() == 0
    for q, kq, vq, Os, ls in outs:
        for b in range(w.batch):
            out, l2, Kc_ref[b], Vc_ref[b], n2 = O.attention(Kc_ref[b], Vc_ref[b], n, to_f64(q[b]), to_f64(kq[b]),
                                                            to_f64(vq[b]))
            assert np.abs(to_f64(Os[b]) - out).max() <= 2e-2
            assert np.abs(to_f64(ls[b]) - l2).max() <= 2e-2
        n += 64
    assert run.cache_len.cpu().tolist() == [[n] * w.batch]
    for b in range(w.batch):
        out, l2, _, _, _ = O.attention(Kc_ref[b], Vc_ref[b], n, to_f64(q_last[b]))
        assert np.abs(to_f64(O_last[b]) - out).max() <= 2e-2
        assert np.abs(to_f64(lse_last[b]) - l2).max() <= 2e-2
        assert np.array_equal(to_f64(run.Kc[0, b])[:, :n], Kc_ref[b][:, :n])


@pytest.mark.parametrize("case", ["cfg0", "cfg1", "ragged_f32", "ragged_bf16_d64", "blocks16", "paper_blocks", "all_kept",
                                  "protected_only"])
def test_sparsify_in_one_call_equals_the_three_calls(case):
    """samkv_sparsify (score, then selection and gather fused in one launch) and samkv_select_compact write exactly
    what samkv_score + samkv_select + samkv_compact write: scores, unit list, compact cache, cache length and inverse
    map, bit for bit."""
    k_units = None
    if case in ("cfg0", "cfg1"):
        w = synth.CONFIGS[case]
    elif case == "ragged_f32":
        w = synth.ragged_workload(dtype="f32", head_dim=64)
    elif case == "ragged_bf16_d64":
        w = synth.ragged_workload(dtype="bf16", head_dim=64, n_q_heads=8, n_kv_heads=2)
    elif case == "blocks16":
        w = synth.ragged_workload(ctx_lens=(160, 257, 64, 1000), dtype="bf16", head_dim=128, block_size=16, n_init=16, n_local=32)
    elif case == "paper_blocks":
        w = synth.CONFIGS["cfg1"].replace(block_size=64, n_init=64, n_local=128)
    else:
        w = synth.ragged_workload(dtype="bf16", head_dim=128)
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    shape = B.Shape.from_workload(w)
    if case == "all_kept":
        prot, U_tot, _ = B.samkv_layout(shape)
        k_units = [-(-n // w.block_size) for n in w.ctx_lens]
    elif case == "protected_only":
        k_units = list(B.samkv_layout(shape)[0])
    ref = DeviceRun(w, inp, k_units=k_units).sparsify()
    torch.cuda.synchronize()
    for fused_score in (True, False):
        got = DeviceRun(w, inp, k_units=k_units)
        got.Kc.fill_(7.0); got.Vc.fill_(7.0); got.inv_map.fill_(123)
        ref2 = DeviceRun(w, inp, k_units=k_units)
        ref2.Kc.fill_(7.0); ref2.Vc.fill_(7.0); ref2.inv_map.fill_(123)
        ref2.sparsify()
        if fused_score:
            B.samkv_sparsify(got.handle, got.shape, inp["K"], inp["V"], inp["Q"], w.q_tokens, inp["Qloc"],
                             inp["Qloc"].shape[3], 1, got.k_units, got.scores, got.sel, got.Kc, got.Vc, got.capacity,
                             got.cache_len, got.inv_map)
        else:
            B.samkv_select_compact(got.handle, got.shape, ref.scores, got.k_units, inp["K"], inp["V"], got.sel, got.Kc,
                                   got.Vc, got.capacity, got.cache_len, got.inv_map)
        torch.cuda.synchronize()
        assert got.poll() == 0
        if fused_score:
            assert torch.equal(got.scores, ref2.scores)
        assert torch.equal(got.sel, ref2.sel)
        assert torch.equal(got.cache_len, ref2.cache_len)
        assert torch.equal(got.inv_map, ref2.inv_map)
        view = torch.int16 if w.dtype == "bf16" else torch.int32
        assert torch.equal(got.Kc.view(view), ref2.Kc.view(view))       # untouched tail slots included
        assert torch.equal(got.Vc.view(view), ref2.Vc.view(view))


def test_sparsify_refuses_bad_arguments_before_launching_anything():
    w = synth.CONFIGS["cfg0"]
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp)
    run.scores.fill_(-3.0)
    with pytest.raises(B.SamkvError) as e:
        B.samkv_sparsify(run.handle, run.shape, inp["K"], inp["V"], inp["Q"], w.q_tokens, inp["Qloc"], inp["Qloc"].shape[3],
                         1, run.k_units, run.scores, run.sel, run.Kc, run.Vc, run.S - 1, run.cache_len, run.inv_map)
    assert e.value.status == 4                                            # capacity
    with pytest.raises(B.SamkvError) as e:
        B.samkv_sparsify(run.handle, run.shape, inp["K"], inp["V"], inp["Q"], w.q_tokens, inp["Qloc"], inp["Qloc"].shape[3],
                         1, [10 ** 6] * w.n_ctx, run.scores, run.sel, run.Kc, run.Vc, run.capacity, run.cache_len,
                         run.inv_map)
    assert e.value.status == 5                                            # budget
    torch.cuda.synchronize()
    assert bool((run.scores == -3.0).all())                               # the scoring step was not enqueued either


@pytest.mark.parametrize("long_kv", [False, True])
def test_attention_sees_q_written_by_the_kernel_right_before_it(long_kv):
    """Stream order on Q: a kernel on the same stream writes Q immediately before every one of several hundred
    back-to-back attention calls on the tensor-memory path (which is launched as a programmatic dependent and
    overlaps its set-up with the kernel before it).  Every output must equal the output for that Q computed after
    a full synchronisation, and those reference outputs are checked against the oracle.  long_kv: one layer buffer
    of the stress configuration at full budget, which takes the 256-row kernel (its oracle parity is covered by the
    budget sweep of the full-size tests; here only the order is checked)."""
    w = synth.CONFIGS["cfg4"].replace(budget_bp=10000) if long_kv else synth.CONFIGS["cfg1"]
    inp = synth.make_inputs(w, DEV) if long_kv else {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp).sparsify()
    torch.cuda.synchronize()
    g = torch.Generator(device=DEV).manual_seed(5)
    n_src, n_calls = (4, 48) if long_kv else (4, 320)
    Q_src = torch.randn((n_src,) + tuple(inp["Qa"][0].shape), generator=g, device=DEV).to(w.torch_dtype)
    Kc0, Vc0 = run.Kc[0].clone(), run.Vc[0].clone()
    for with_chunk in (False, True):
        Kq = inp["Kq"][0] if with_chunk else None
        Vq = inp["Vq"][0] if with_chunk else None
        refs = []
        for i in range(n_src):                                # references: everything complete before the call
            run.cache_len.fill_(run.S)
            torch.cuda.synchronize()
            Oref, lse = run.attn(0, Q_src[i].clone(), Kq, Vq)
            torch.cuda.synchronize()
            if not long_kv:
                check_attention(w, Kc0[0], Vc0[0], run.S, Q_src[i][0], None if Kq is None else Kq[0],
                                None if Vq is None else Vq[0], Oref[0], lse[0])
            refs.append(Oref)
        Q = torch.empty_like(Q_src[0])
        outs = torch.empty((n_calls,) + tuple(Q.shape), dtype=Q.dtype, device=DEV)
        for i in range(n_calls):                              # no host synchronisation in this loop
            if with_chunk:
                run.cache_len.fill_(run.S)
            Q.copy_(Q_src[i % n_src])                         # the producer of Q: a kernel on the same stream
            B.samkv_attn(run.handle, run.shape, 0, run.Kc, run.Vc, run.capacity, run.cache_len, Q, w.q_tokens, Kq, Vq,
                         0.0, outs[i], None)
        torch.cuda.synchronize()
        assert run.poll() == 0
        for i in range(n_calls):
            assert torch.equal(outs[i], refs[i % n_src]), f"call {i} (chunk appended: {with_chunk}) read a stale Q"


def test_a_five_percent_error_in_attention_would_be_caught():
    """The relative bound bites on N(0,1) data: the library's own cfg1 output, scaled by 1.05, fails it."""
    import samkv_testlib as T
    w = synth.CONFIGS["cfg1"]
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp).sparsify()
    Kc0, Vc0 = run.Kc[0].clone(), run.Vc[0].clone()
    Og, lse = run.attn(0, inp["Qa"][0], inp["Kq"][0], inp["Vq"][0])
    torch.cuda.synchronize()
    T.OBSERVED["attn_rel"] = 0.0
    check_attention(w, Kc0[0], Vc0[0], run.S, inp["Qa"][0, 0], inp["Kq"][0, 0], inp["Vq"][0, 0], Og[0], lse[0])
    print(f"cfg1 attention: largest error {T.OBSERVED['attn_rel']:.3e} of a head's largest output, lse {T.OBSERVED['lse']:.3e}")
    with pytest.raises(AssertionError):
        check_attention(w, Kc0[0], Vc0[0], run.S, inp["Qa"][0, 0], inp["Kq"][0, 0], inp["Vq"][0, 0],
                        (Og[0].float() * 1.05).to(Og.dtype), lse[0])


@pytest.mark.parametrize("ctx_lens,T_q,Hq,Hkv,budget_bp", [
    ((40, 30), 32, 8, 2, 10000),          # 128 rows, one partial KV tile: cache (70) + chunk (32) < 128 slots
    ((100, 90), 129, 2, 2, 10000),        # G = 1, 129 rows: a second query tile with a single real row
    ((200, 56), 16, 32, 2, 10000),        # G = 16, 256 rows; the chunk crosses the 256-slot tile boundary
    ((700, 900, 333), 50, 12, 2, 3000),   # G = 6 (rows of one token straddle lane quarters), 300 rows, ragged
    ((2048,) * 3, 128, 16, 2, 10000),     # 1024 rows per KV head: eight query tiles share each K/V tile
])
def test_tensor_memory_attention_edge_shapes(ctx_lens, T_q, Hq, Hkv, budget_bp):
    """Shapes that exercise the tcgen05 kernels' corners: partial tiles, single-row query tiles, large groups."""
    w = synth.ragged_workload(ctx_lens=ctx_lens, dtype="bf16", head_dim=128, n_q_heads=Hq, n_kv_heads=Hkv,
                              q_tokens=T_q, n_init=4, n_local=8, budget_bp=budget_bp, seed=1234 + T_q)
    full_check(w)


@pytest.mark.parametrize("dtype,T_q,Hq,n,share", [("bf16", 64, 8, 3, False), ("bf16", 64, 8, 3, True), ("bf16", 32, 8, 2, False),
                                                   ("bf16", 1, 8, 4, False), ("f32", 5, 4, 4, False)])
def test_attention_of_several_layers_in_one_call(dtype, T_q, Hq, n, share):
    """samkv_attn_layers over n of 4 layers (a range that starts at layer 1 where it can): every layer against the
    oracle on its own cache, appended rows bit-exact in their layer's cache, cache lengths bumped for exactly the
    layers of the call; tensor-memory kernels (both), the mma.sync kernel (decode row) and the fp32 kernel."""
    w = synth.ragged_workload(ctx_lens=(700, 900, 333), dtype=dtype, head_dim=128 if dtype == "bf16" else 64,
                              n_q_heads=Hq, n_kv_heads=2, q_tokens=T_q, n_init=4, n_local=8, budget_bp=3000,
                              seed=99 + T_q).replace(n_layers=4, batch=2)
    inp = {k: v.to(DEV) for k, v in synth.make_inputs(w, "cpu").items()}
    run = DeviceRun(w, inp).sparsify()
    torch.cuda.synchronize()
    l0 = 4 - n if n < 4 else 0
    handle = B.Handle(B.Shape.from_workload(w.replace(batch=w.batch * n), n_layers=1), T_q, run.capacity)
    B.samkv_attn_share_sm(handle, share)
    Kc0, Vc0 = run.Kc.clone(), run.Vc.clone()
    sl = slice(l0, l0 + n)
    Og = torch.empty_like(inp["Qa"][sl])
    lse = torch.empty((n, w.batch, Hq, T_q), dtype=torch.float32, device=DEV)
    B.samkv_attn_layers(handle, run.shape, l0, n, run.Kc, run.Vc, run.capacity, run.cache_len, inp["Qa"][sl], T_q,
                        inp["Kq"][sl], inp["Vq"][sl], 0.0, Og, lse)
    torch.cuda.synchronize()
    assert B.samkv_poll_status(handle) == 0
    for i, l in enumerate(range(l0, l0 + n)):
        for b in range(w.batch):
            err, K2, V2, m = check_attention(w, Kc0[l, b], Vc0[l, b], run.S, inp["Qa"][l, b], inp["Kq"][l, b],
                                             inp["Vq"][l, b], Og[i, b], lse[i, b])
            assert np.array_equal(to_f64(run.Kc[l, b][:, run.S:m]), K2[:, run.S:m])
            assert np.array_equal(to_f64(run.Vc[l, b][:, run.S:m]), V2[:, run.S:m])
    want = [[run.S + (T_q if l0 <= l < l0 + n else 0)] * w.batch for l in range(4)]
    assert run.cache_len.cpu().tolist() == want
    untouched = [l for l in range(4) if not (l0 <= l < l0 + n)]
    for l in untouched:
        assert torch.equal(run.Kc[l], Kc0[l]) and torch.equal(run.Vc[l], Vc0[l])
    for bad_l0, bad_n in ((-1, 1), (0, 0), (3, 2), (0, 5)):                      # ranges outside the cache: refused
        with pytest.raises(B.SamkvError) as e:
            B.samkv_attn_layers(handle, run.shape, bad_l0, bad_n, run.Kc, run.Vc, run.capacity, run.cache_len,
                                inp["Qa"][sl], T_q, None, None, 0.0, Og, None)
        assert e.value.status == 1
    assert run.poll() == 0


@pytest.fixture
def attention_shares_its_sm():
    import samkv_testlib as T
    T.ATTN_SHARE_SM = True
    yield
    T.ATTN_SHARE_SM = False


SHARE_CASES = {
    "cfg1": lambda: test_cfg1_llama_shape_bf16(),
    "chunks": lambda: test_chunked_prefill_on_the_tensor_memory_kernel(),
    "stream_order_on_q": lambda: test_attention_sees_q_written_by_the_kernel_right_before_it(False),
    "rows_160_many_splits": lambda: test_attention_row_tilings_and_long_cache(40, 4),
    "rows_512_many_splits": lambda: test_attention_row_tilings_and_long_cache(64, 8),
    "partial_tile": lambda: test_tensor_memory_attention_edge_shapes((40, 30), 32, 8, 2, 10000),
    "single_row_tile": lambda: test_tensor_memory_attention_edge_shapes((100, 90), 129, 2, 2, 10000),
    "g16": lambda: test_tensor_memory_attention_edge_shapes((200, 56), 16, 32, 2, 10000),
    "g6_ragged": lambda: test_tensor_memory_attention_edge_shapes((700, 900, 333), 50, 12, 2, 3000),
    "perturbation": lambda: test_a_five_percent_error_in_attention_would_be_caught(),
}


@pytest.mark.parametrize("case", sorted(SHARE_CASES))
def test_attention_kernel_that_leaves_room_on_its_sm(case, attention_shares_its_sm):
    """samkv_attn_share_sm(handle, 1) routes bf16 prefill chunks to the double-buffered 128-row kernel (with the
    separate append and merge launches where it needs them); the same cases and bounds as for the default kernel."""
    SHARE_CASES[case]()


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_against_the_oracle(seed):
    """Seeded random small workloads: every stage of the path against the oracle (shapes no hand-written case covers)."""
    r = np.random.default_rng(9000 + seed)
    Bsz = int(2 ** r.integers(0, 5))                                   # block size 1 .. 16
    n_ctx = int(r.integers(1, 7))
    lens = tuple(int(x) for x in r.integers(3 * Bsz + 1, 40 * Bsz + 200, size=n_ctx))
    G = int(r.choice([1, 2, 4, 8]))
    Hkv = int(r.choice([1, 2, 4]))
    dtype = str(r.choice(["bf16", "f32"]))
    d = int(r.choice([64, 128]))
    T_q = int(r.integers(1, 70))
    n_init = Bsz * int(r.integers(0, 3))
    n_local = Bsz * int(r.integers(1, 4))
    w = synth.ragged_workload(name=f"fuzz{seed}", ctx_lens=lens, dtype=dtype, head_dim=d, n_q_heads=G * Hkv,
                              n_kv_heads=Hkv, q_tokens=T_q, block_size=Bsz, n_init=n_init, n_local=n_local,
                              budget_bp=int(r.integers(500, 10001)), seed=9000 + seed)
    w = w.replace(n_layers=int(r.integers(1, 3)), batch=int(r.integers(1, 3)))
    full_check(w)

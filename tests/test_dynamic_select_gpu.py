"""GPU parity of the paper's dynamic selection: Top-P per document (Eq. 2, Eq. 3), the cross-context
Top-K over the retrieved blocks (Sec. 3.2), and the gather of the resulting unit lists.

The oracle is fed the library's own fp32 scores (their parity is covered elsewhere), so every
comparison here isolates the selection arithmetic.  Rules:
  * P: |P_gpu - P_oracle| <= 2e-5 (fp32 anchor sums against fp64; P lies in [0, 1]).
  * candidate counts, K, S_u, kept tokens: equal to the oracle's on the SAME P values.
  * unit lists: equal to the oracle's except at units whose normalised score (fp64) lies within
    1e-6 of the oracle's K-th normalised score, the kernel normalising in fp32; lists are ascending,
    of the stated length, and contain every protected unit.
  * compaction: bit-exact gather of the GPU's own list; inverse-map round trip."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import samkv_oracle as O
from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import synth
from samkv_testlib import DeviceRun

pytestmark = pytest.mark.gpu


def gpu_scores(w, scores=None):
    inp = synth.make_inputs(w, "cuda")
    run = DeviceRun(w, inp)
    if scores is None:
        B.samkv_score(run.handle, run.shape, inp["K"], inp["Q"], w.q_tokens, inp["Qloc"], inp["Qloc"].shape[3], 1,
                      run.scores, run.qhat)
    else:
        run.scores.copy_(scores)
    torch.cuda.synchronize()
    return run, inp


def oracle_P(w, u_all, star, max_units=None, min_units=None):
    """u_all: [L, Bt, Hkv, U_tot] float64 -> P [Bt, D]."""
    out = []
    for b in range(w.batch):
        P_layers = np.stack([
            O.top_p_per_head(u_all[l, b], w.ctx_offsets, w.block_size, w.n_init, w.n_local,
                             None if max_units is None else max_units[l, b],
                             None if min_units is None else min_units[l, b]) for l in star])
        out.append(O.consolidate_top_p(P_layers))
    return np.stack(out)


def normalised(w, u_row):
    """fp64 min-max normalised middle-unit scores of one head, indexed by global unit id (NaN elsewhere)."""
    nb, off = O.unit_layout(w.ctx_offsets, w.block_size)
    v = np.full(u_row.shape[0], np.nan)
    for c in range(w.n_ctx):
        mid = O.middle_units(w.ctx_lens[c], w.block_size, w.n_init, w.n_local)
        if not mid:
            continue
        ids = np.array([off[c] + m for m in mid])
        lo, hi = u_row[ids].min(), u_row[ids].max()
        v[ids] = (u_row[ids] - lo) / (hi - lo) if hi > lo else 0.0
    return v


def check_cross(w, u, cand, sel_gpu, counts_gpu, where=""):
    """u [Hkv, U_tot] fp64, sel_gpu [Hkv, S_u], counts_gpu [Hkv, D].  Returns the number of heads that differed."""
    sel_or, counts_or = O.cross_context_select(u, w.ctx_offsets, w.block_size, w.n_init, w.n_local, cand)
    assert sel_gpu.shape == sel_or.shape, f"{where}: list length {sel_gpu.shape} vs {sel_or.shape}"
    nb, off = O.unit_layout(w.ctx_offsets, w.block_size)
    prot = set()
    for c in range(w.n_ctx):
        prot |= set(off[c] + m for m in O.protected_units(w.ctx_lens[c], w.block_size, w.n_init, w.n_local))
    K = sum(cand) // w.n_ctx
    n_diff = 0
    for h in range(u.shape[0]):
        g, o = sel_gpu[h], sel_or[h]
        assert np.all(np.diff(g) > 0), f"{where} h{h}: ids not strictly ascending"
        assert g.min() >= 0 and g.max() < off[-1]
        assert prot <= set(g.tolist()), f"{where} h{h}: protected unit missing"
        # counts must describe the GPU's own list
        own = np.array([np.sum((g >= off[c]) & (g < off[c + 1])) for c in range(w.n_ctx)])
        assert np.array_equal(own, counts_gpu[h]), f"{where} h{h}: counts do not match the list"
        if np.array_equal(g, o):
            assert np.array_equal(counts_gpu[h], counts_or[h])
            continue
        n_diff += 1
        v = normalised(w, u[h])
        chosen_or = sorted(set(o.tolist()) - prot, key=lambda uid: (-v[uid], uid))
        v_K = v[chosen_or[K - 1]]
        for uid in set(g.tolist()) ^ set(o.tolist()):
            assert abs(v[uid] - v_K) <= 1e-6, (f"{where} h{h}: unit {uid} differs outside the tie band "
                                               f"(normalised {v[uid]}, K-th {v_K})")
        # every unit the GPU kept must have been retrieved by its own document (exact stage, fp32 keys)
        for c in range(w.n_ctx):
            mid = O.middle_units(w.ctx_lens[c], w.block_size, w.n_init, w.n_local)
            order = sorted(mid, key=lambda m: (-u[h, off[c] + m], m))[: cand[c]]
            retrieved = set(off[c] + m for m in order)
            mine = set(x for x in g.tolist() if off[c] <= x < off[c + 1]) - prot
            assert mine <= retrieved, f"{where} h{h} c{c}: kept a unit its document did not retrieve"
    return n_diff


def check_compact_units(w, inp, l, b, sel_lb, Kc, Vc, inv, cache_len, S):
    K = inp["K"][l, b].cpu()
    V = inp["V"][l, b].cpu()
    assert int(cache_len[l, b]) == S
    for h in range(w.n_kv_heads):
        toks = O.units_to_tokens(sel_lb[h], w.ctx_offsets, w.block_size)
        assert len(toks) == S
        idx = torch.from_numpy(toks)
        assert torch.equal(Kc[l, b, h, :S].cpu().view(torch.uint8), K[h, idx].view(torch.uint8)), f"Kc l{l} b{b} h{h}"
        assert torch.equal(Vc[l, b, h, :S].cpu().view(torch.uint8), V[h, idx].view(torch.uint8)), f"Vc l{l} b{b} h{h}"
        exp = np.full(w.l_tot, -1, dtype=np.int32)
        exp[toks] = np.arange(S, dtype=np.int32)
        assert np.array_equal(inv[l, b, h].cpu().numpy(), exp), f"inv_map l{l} b{b} h{h}"
    assert not Kc[l, b, :, S:].float().any() and not Vc[l, b, :, S:].float().any()


def run_dynamic(w, star=None, scores=None, with_blocks=False, P_override=None, compact=True):
    """Whole dynamic path on one workload; returns (P_gpu, cand, K, number of heads that differed)."""
    run, inp = gpu_scores(w, scores)
    dev = run.scores.device
    L, Bt, Hkv, D = w.n_layers, w.batch, w.n_kv_heads, w.n_ctx
    star = list(range(L)) if star is None else star
    u_all = run.scores.cpu().double().numpy()
    nb, off = O.unit_layout(w.ctx_offsets, w.block_size)
    max_u = min_u = None
    if with_blocks:                                            # stand-in for the offline analysis: any middle unit
        rng = np.random.default_rng(w.seed)
        max_u = np.zeros((L, Bt, D), dtype=np.int32)
        min_u = np.zeros((L, Bt, D), dtype=np.int32)
        for c in range(D):
            mid = O.middle_units(w.ctx_lens[c], w.block_size, w.n_init, w.n_local) or [0]
            max_u[:, :, c] = off[c] + rng.choice(mid, size=(L, Bt))
            min_u[:, :, c] = off[c] + rng.choice(mid, size=(L, Bt))
    P_gpu = torch.full((Bt, D), -1.0, dtype=torch.float32, device=dev)
    B.samkv_topp(run.handle, run.shape, run.scores, star,
                 None if max_u is None else torch.from_numpy(max_u).to(dev),
                 None if min_u is None else torch.from_numpy(min_u).to(dev), P_gpu)
    torch.cuda.synchronize()
    P_gpu = P_gpu.cpu().numpy()
    P_or = oracle_P(w, u_all, star, max_u, min_u)
    assert np.abs(P_gpu - P_or).max() <= 2e-5, f"P mismatch: {np.abs(P_gpu - P_or).max()}"
    assert P_gpu.min() >= 0.0 and P_gpu.max() <= 1.0

    # the request's ratios are those of batch element 0 (the candidate counts are shared by the batch)
    P_row = P_gpu[0] if P_override is None else np.asarray(P_override, dtype=np.float32)
    cand, K, S_u, S = B.samkv_topp_plan(run.shape, [float(x) for x in P_row])
    cand_or = O.candidate_counts(P_row.astype(np.float64), w.ctx_offsets, w.block_size, w.n_init, w.n_local)
    assert cand == cand_or
    assert K == sum(cand) // D
    n_prot = sum(len(O.protected_units(n, w.block_size, w.n_init, w.n_local)) for n in w.ctx_lens)
    assert S_u == n_prot + K

    sel = torch.full((L, Bt, Hkv, S_u), -7, dtype=torch.int32, device=dev)
    counts = torch.full((L, Bt, Hkv, D), -7, dtype=torch.int32, device=dev)
    n_scratch = B.samkv_select_cross_scratch_bytes(run.shape, cand)
    assert n_scratch <= B.samkv_select_cross_scratch_bytes(run.shape)
    scratch = torch.empty(n_scratch, dtype=torch.uint8, device=dev)
    B.samkv_select_cross(run.handle, run.shape, run.scores, cand, scratch, sel, counts)
    torch.cuda.synchronize()
    sel_np, counts_np = sel.cpu().numpy(), counts.cpu().numpy()
    n_diff = 0
    for l in range(L):
        for b in range(Bt):
            n_diff += check_cross(w, u_all[l, b], cand, sel_np[l, b], counts_np[l, b], where=f"l{l} b{b}")
    assert S == len(O.units_to_tokens(sel_np[0, 0, 0], w.ctx_offsets, w.block_size))

    if compact:
        cap = S + 3
        Kc = torch.zeros((L, Bt, Hkv, cap, w.head_dim), dtype=w.torch_dtype, device=dev)
        Vc = torch.zeros_like(Kc)
        cache_len = torch.zeros((L, Bt), dtype=torch.int32, device=dev)
        inv = torch.zeros((L, Bt, Hkv, w.l_tot), dtype=torch.int32, device=dev)
        B.samkv_compact_units(run.handle, run.shape, inp["K"], inp["V"], sel, S_u, Kc, Vc, cap, cache_len, inv)
        torch.cuda.synchronize()
        assert run.poll() == 0
        for l in sorted({0, L - 1}):
            for b in sorted({0, Bt - 1}):
                check_compact_units(w, inp, l, b, sel_np[l, b], Kc, Vc, inv, cache_len, S)
    return P_gpu, cand, K, n_diff, sel_np, counts_np


# ------------------------------------------------------------------------------------------- cases
def test_dynamic_cfg0_token_units():
    w = synth.CONFIGS["cfg0"]
    P, cand, K, _, sel, counts = run_dynamic(w)
    assert K > 0


def test_dynamic_cfg1_bf16():
    w = synth.CONFIGS["cfg1"]
    P, cand, K, _, sel, counts = run_dynamic(w)
    assert K > 0
    # the split between documents is free: some head must deviate from an even split
    mid_counts = counts[0, 0] - counts[0, 0].min(axis=0, keepdims=True)
    assert mid_counts.any()


@pytest.mark.parametrize("block_size,n_init,n_local", [(16, 16, 32), (64, 64, 64), (4, 0, 4)])
def test_dynamic_block_units_ragged(block_size, n_init, n_local):
    w = synth.ragged_workload(ctx_lens=(1000, 257, 4099, 700, 64 * 3 + 5), block_size=block_size, n_init=n_init,
                              n_local=n_local, seed=500 + block_size)
    run_dynamic(w)


def test_dynamic_multi_layer_batch_star_subset():
    w = dataclasses.replace(synth.CONFIGS["cfg1"], name="dyn_lb", n_layers=5, batch=3, ctx_lens=(512, 768, 300, 1024),
                            seed=321)
    run_dynamic(w, star=[1, 3, 4])


def test_dynamic_caller_max_min_blocks():
    w = dataclasses.replace(synth.CONFIGS["cfg1"], name="dyn_blocks", n_layers=3, batch=2, block_size=16, n_init=16,
                            n_local=32, ctx_lens=(1024, 777, 1536), seed=322)
    run_dynamic(w, with_blocks=True)


@pytest.mark.parametrize("P_row", [[0.0, 0.0, 0.0, 0.0], [1.0, 1.0, 1.0, 1.0], [1.0, 0.0, 0.0, 0.0],
                                   [0.001, 0.5, 0.0, 0.25]])
def test_dynamic_ratio_edges(P_row):
    """P = 0 everywhere keeps the protected units only; P = 1 everywhere retrieves every middle unit and keeps
    K = their mean count per document; a single document with candidates feeds all K places."""
    w = synth.ragged_workload(ctx_lens=(300, 257, 640, 100), block_size=4, n_init=4, n_local=8, seed=91)
    P, cand, K, _, sel, counts = run_dynamic(w, P_override=P_row)
    if not any(P_row):
        assert K == 0
    if P_row == [1.0, 0.0, 0.0, 0.0]:
        assert (counts[..., 1:] == np.array([len(O.protected_units(n, 4, 4, 8)) for n in w.ctx_lens[1:]])).all()


def test_dynamic_ties_constant_scores():
    """All scores equal: every normalised score is 0, so the K lowest retrieved global ids win."""
    w = synth.ragged_workload(ctx_lens=(200, 120, 333), block_size=1, n_init=4, n_local=8, seed=92)
    shape = B.Shape.from_workload(w)
    prot, U_tot, _ = B.samkv_layout(shape, B.samkv_budget_units(shape, w.budget_bp))
    scores = torch.full((1, 1, w.n_kv_heads, U_tot), 1.25, dtype=torch.float32, device="cuda")
    P, cand, K, n_diff, sel, counts = run_dynamic(w, scores=scores, P_override=[0.5, 0.25, 0.75])
    assert n_diff == 0
    assert P.max() == 0.0                    # s_anc == s_max == s_min: not inside (s_min, s_max]


def test_dynamic_ties_quantised_scores():
    """Scores on a coarse grid: many exact ties inside documents (lower index wins) and, after normalisation,
    across documents (lower global id wins)."""
    w = synth.ragged_workload(ctx_lens=(500, 500, 500, 260), block_size=1, n_init=4, n_local=8, seed=93)
    shape = B.Shape.from_workload(w)
    prot, U_tot, _ = B.samkv_layout(shape, B.samkv_budget_units(shape, w.budget_bp))
    g = torch.Generator(device="cuda").manual_seed(93)
    scores = torch.randint(0, 9, (1, 1, w.n_kv_heads, U_tot), generator=g, device="cuda").float() * 0.5 - 1.0
    P, cand, K, n_diff, sel, counts = run_dynamic(w, scores=scores, P_override=[0.3, 0.3, 0.3, 0.3])
    assert n_diff == 0       # equal inputs give equal quotients in either precision; distinct grid values stay apart


def test_dynamic_bench_shape_slab_sample():
    """cfg2's shape (20 documents of 1536 tokens, token units) on a few layers."""
    w = dataclasses.replace(synth.CONFIGS["cfg2"], name="dyn_cfg2", n_layers=2, batch=2)
    run_dynamic(w)


def test_dynamic_errors():
    w = synth.CONFIGS["cfg0"]
    run, inp = gpu_scores(w)
    P = torch.zeros((1, w.n_ctx), dtype=torch.float32, device="cuda")
    with pytest.raises(B.SamkvError):
        B.samkv_topp(run.handle, run.shape, run.scores, [], None, None, P)            # no stable layer
    with pytest.raises(B.SamkvError):
        B.samkv_topp(run.handle, run.shape, run.scores, [w.n_layers], None, None, P)  # layer out of range
    with pytest.raises(B.SamkvError):
        B.samkv_topp_plan(run.shape, [1.5] + [0.0] * (w.n_ctx - 1))
    with pytest.raises(B.SamkvError):
        B.samkv_topp_plan(run.shape, [float("nan")] + [0.0] * (w.n_ctx - 1))
    sel = torch.zeros((1, 1, w.n_kv_heads, 4096), dtype=torch.int32, device="cuda")
    scratch = torch.empty(B.samkv_select_cross_scratch_bytes(run.shape), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SamkvError):
        B.samkv_select_cross(run.handle, run.shape, run.scores, [10 ** 6] + [0] * (w.n_ctx - 1), scratch, sel)
    with pytest.raises(B.SamkvError):                                                  # scratch too small
        B.samkv_select_cross(run.handle, run.shape, run.scores, [1] * w.n_ctx, scratch[:16], sel)
    assert run.poll() == 0


def test_dynamic_end_to_end_attention():
    """Scores -> Top-P -> cross-context Top-K -> gather -> attention with the query chunk appended: the output must
    equal the oracle's attention over the oracle's gather of the same unit lists."""
    from samkv_testlib import check_attention, to_f64
    w = synth.CONFIGS["cfg1"]
    run, inp = gpu_scores(w)
    dev = run.scores.device
    L, Bt, Hkv, D = w.n_layers, w.batch, w.n_kv_heads, w.n_ctx
    P = torch.zeros((Bt, D), dtype=torch.float32, device=dev)
    B.samkv_topp(run.handle, run.shape, run.scores, [0], None, None, P)
    cand, K, S_u, S = B.samkv_topp_plan(run.shape, [float(x) for x in P[0].cpu()])
    assert S + w.q_tokens <= run.capacity
    sel = torch.zeros((L, Bt, Hkv, S_u), dtype=torch.int32, device=dev)
    scratch = torch.empty(B.samkv_select_cross_scratch_bytes(run.shape, cand), dtype=torch.uint8, device=dev)
    B.samkv_select_cross(run.handle, run.shape, run.scores, cand, scratch, sel)
    B.samkv_compact_units(run.handle, run.shape, inp["K"], inp["V"], sel, S_u, run.Kc, run.Vc, run.capacity,
                          run.cache_len, run.inv_map)
    torch.cuda.synchronize()
    sel_np = sel.cpu().numpy()
    Kc_or, Vc_or, S_or, inv_or = O.compact(inp["K"][0, 0].cpu().float().numpy(), inp["V"][0, 0].cpu().float().numpy(),
                                           sel_np[0, 0], w.ctx_offsets, w.block_size, capacity=S + w.q_tokens)
    assert S_or == S and int(run.cache_len[0, 0]) == S
    assert np.array_equal(inv_or, run.inv_map[0, 0].cpu().numpy())
    Og, lse = run.attn(0, inp["Qa"][0], inp["Kq"][0], inp["Vq"][0])
    torch.cuda.synchronize()
    assert run.poll() == 0
    assert int(run.cache_len[0, 0]) == S + w.q_tokens
    check_attention(w, torch.from_numpy(Kc_or), torch.from_numpy(Vc_or), S, inp["Qa"][0, 0], inp["Kq"][0, 0],
                    inp["Vq"][0, 0], Og[0], lse[0])


@pytest.mark.parametrize("seed", range(12))
def test_dynamic_random_shapes(seed):
    """Seeded random small workloads through Top-P, cross-context Top-K and the gather of its unit lists."""
    r = np.random.default_rng(7000 + seed)
    Bsz = int(2 ** r.integers(0, 5))
    n_ctx = int(r.integers(1, 7))
    lens = tuple(int(x) for x in r.integers(3 * Bsz + 1, 40 * Bsz + 300, size=n_ctx))
    Hkv = int(r.choice([1, 2, 4]))
    w = synth.ragged_workload(name=f"dynfuzz{seed}", ctx_lens=lens, dtype=str(r.choice(["bf16", "f32"])),
                              head_dim=int(r.choice([64, 128])), n_q_heads=2 * Hkv, n_kv_heads=Hkv,
                              q_tokens=int(r.integers(1, 20)), block_size=Bsz, n_init=Bsz * int(r.integers(0, 3)),
                              n_local=Bsz * int(r.integers(1, 4)), seed=7000 + seed)
    w = dataclasses.replace(w, n_layers=int(r.integers(1, 4)), batch=int(r.integers(1, 3)))
    P_override = None if seed % 2 == 0 else [float(x) for x in r.random(n_ctx)]
    run_dynamic(w, star=list(range(w.n_layers))[-2:], P_override=P_override)

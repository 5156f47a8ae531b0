"""Block representatives (Sec. 3.2): mean key per unit, and scoring on the representatives.

Rules:
  * Kbar: |Kbar_gpu - exact fp64 mean| <= half an ulp of the storage type + 2e-6 * mean |k| of the unit (fp32
    accumulation in another order than the oracle's); where the oracle's rounded value differs, that is a tie at the
    rounding boundary.
  * scores on the representatives: against the oracle's inner products with the GPU's own Kbar values, with the
    bound used for token scores (1e-5 * |q| * max|Kbar row|).
  * against the block mean of the token scores (the quantity the representatives stand for) the deviation is the
    storage rounding of Kbar: <= 2^-8 * |q|_1-weighted bound, checked loosely as 1e-2 * |q| * max|Kbar row| for bf16."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import samkv_oracle as O
from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import synth
from samkv_testlib import DeviceRun, oracle_scores, to_f64, check_selection

pytestmark = pytest.mark.gpu


def ulp(x, dtype):
    e = np.floor(np.log2(np.maximum(np.abs(x), 1e-300)))
    return 2.0 ** (e - (7 if dtype == "bf16" else 23))


def block_run(w):
    inp = synth.make_inputs(w, "cuda")
    run = DeviceRun(w, inp)
    Kbar = torch.full((w.n_layers, w.batch, w.n_kv_heads, run.U_tot, w.head_dim), 7.0, dtype=w.torch_dtype, device="cuda")
    B.samkv_block_means(run.handle, run.shape, inp["K"], Kbar)
    scores = torch.full_like(run.scores, -5.0)
    B.samkv_score_blocks(run.handle, run.shape, Kbar, inp["Q"], w.q_tokens, inp["Qloc"], inp["Qloc"].shape[3], 1, scores,
                         run.qhat)
    torch.cuda.synchronize()
    assert run.poll() == 0
    return run, inp, Kbar, scores


CASES = [
    ("cfg0", dict(block_size=4, n_init=4, n_local=8)),
    ("cfg1", dict(block_size=64, n_init=64, n_local=128)),
    ("cfg1", dict(block_size=16, n_init=16, n_local=32, n_layers=2, batch=2)),
    ("ragged", dict(ctx_lens=(100, 257, 64, 1000, 9), block_size=8, n_init=8, n_local=16)),
    ("ragged", dict(ctx_lens=(130, 77), block_size=32, n_init=32, n_local=32, dtype="bf16", head_dim=64)),
    ("ragged", dict(ctx_lens=(130, 77), block_size=2, n_init=2, n_local=2, dtype="f32", head_dim=128,
                    n_q_heads=8, n_kv_heads=2)),
    ("cfg0", dict(block_size=1)),
]


@pytest.mark.parametrize("name,kw", CASES)
def test_block_means_and_block_scores(name, kw):
    w = dataclasses.replace(synth.CONFIGS[name], **kw) if name in synth.CONFIGS else synth.ragged_workload(**kw)
    run, inp, Kbar, scores = block_run(w)
    nb, unit_off = O.unit_layout(w.ctx_offsets, w.block_size)
    for l in sorted({0, w.n_layers - 1}):
        for b in sorted({0, w.batch - 1}):
            K64 = to_f64(inp["K"][l, b])
            exact = O.block_means(K64, w.ctx_offsets, w.block_size)
            got = to_f64(Kbar[l, b])
            scale = np.abs(K64).mean()
            tol = 0.5 * ulp(exact, w.dtype) + 2e-6 * scale
            assert (np.abs(got - exact) <= tol).all(), f"Kbar l{l} b{b}: {np.abs(got - exact).max()}"
            if w.dtype == "bf16":                                    # fp32 summation error << bf16 ulp: the rounded
                n_off = np.count_nonzero(got != O.block_means(K64, w.ctx_offsets, w.block_size, w.dtype))
                assert n_off <= 1e-3 * got.size                      # values agree except at rounding boundaries
            if w.block_size == 1:
                assert np.array_equal(got, K64)
            # scores against the oracle on the GPU's own representatives
            q, _, u_tok = oracle_scores(w, inp, l, b)                 # q [D, Hkv, d]; u_tok = block means of token scores
            u_rep = O.token_scores(q, got, unit_off)
            ug = to_f64(scores[l, b])
            rownorm = np.sqrt((got ** 2).sum(-1)).max(axis=1)        # [Hkv]
            for c in range(w.n_ctx):
                for h in range(w.n_kv_heads):
                    qn = np.linalg.norm(q[c, h])
                    seg = slice(unit_off[c], unit_off[c + 1])
                    assert np.abs(ug[h, seg] - u_rep[h, seg]).max() <= 1e-5 * qn * rownorm[h]
                    lim = (1e-2 if w.dtype == "bf16" else 1e-5) * qn * rownorm[h]
                    assert np.abs(ug[h, seg] - u_tok[h, seg]).max() <= lim


def test_selection_from_block_scores_follows_the_same_rules():
    """Scores from representatives feed samkv_select / samkv_compact unchanged."""
    w = dataclasses.replace(synth.CONFIGS["cfg1"], block_size=16, n_init=16, n_local=32)
    run, inp, Kbar, scores = block_run(w)
    run.scores.copy_(scores)
    B.samkv_select(run.handle, run.shape, run.scores, run.k_units, run.sel)
    torch.cuda.synchronize()
    u = to_f64(scores[0, 0])
    check_selection(w, run.k_units, run.sel[0, 0].cpu().numpy(), u, where="block scores")


def test_block_means_bench_shape_sample():
    """cfg2's token axis with the paper's 64-token blocks, 2 layers: sampled units against the oracle's mean."""
    w = dataclasses.replace(synth.CONFIGS["cfg2"], name="means_cfg2", n_layers=2, batch=2, block_size=64, n_init=64,
                            n_local=64)
    run, inp, Kbar, scores = block_run(w)
    r = np.random.default_rng(0)
    for _ in range(40):
        l, b, h = int(r.integers(2)), int(r.integers(2)), int(r.integers(8))
        uidx = int(r.integers(run.U_tot))
        c, m = divmod(uidx, 1536 // 64)
        t0 = c * 1536 + m * 64
        exact = to_f64(inp["K"][l, b, h, t0:t0 + 64]).mean(axis=0)
        got = to_f64(Kbar[l, b, h, uidx])
        assert (np.abs(got - exact) <= 0.5 * ulp(exact, "bf16") + 1e-5).all()

"""Pins for the CPU oracle: closed forms, invariants, brute force and library special cases.

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong
sign or index, a transposed operand, an off-by-one in a range) makes it fail.  None of
them re-types the oracle's own formula: expected values are hand-derived constants,
algebraic identities, or results of an independent library routine.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import samkv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(12345)


# ----------------------------------------------------------------------------- pooling
def test_pool_constant_rows_and_single_row():
    row = rng.normal(size=(3, 8))
    Q = np.repeat(row[None], 7, axis=0)
    assert np.allclose(O.pool_query(Q), row, atol=1e-15)
    Q1 = rng.normal(size=(1, 3, 8))
    assert np.array_equal(O.pool_query(Q1), Q1[0])


def test_pool_is_mean_over_tokens_not_heads():
    Q = np.zeros((2, 3, 4))
    Q[0, 1, 2] = 4.0          # token 0, head 1, channel 2
    out = O.pool_query(Q)
    assert out.shape == (3, 4)
    assert out[1, 2] == 2.0 and out.sum() == 2.0
    Ql = np.zeros((2, 2, 3, 4))
    Ql[1, 0, 2, 3] = 6.0
    out = O.pool_local(Ql)
    assert out.shape == (2, 3, 4) and out[1, 2, 3] == 3.0 and out.sum() == 3.0


# ----------------------------------------------------------------------------- Eq. 1
def test_eq1_hand_value_from_golden():
    # tests/golden/eq1_hand_case.txt: D=2, d=2, Q_que=(1,0), q_loc_2=(1,1) => Q^_1=(1+1/sqrt2, 1/sqrt2)
    vals = {}
    with open(os.path.join(GOLDEN, "eq1_hand_case.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split("=")
            vals[k.strip()] = [float(x) for x in v.split(",")]
    Q_que = np.array([vals["Q_que"]])
    q_loc = np.array([[vals["q_loc_1"]], [vals["q_loc_2"]]])
    Qhat = O.personalized_query(Q_que, q_loc)
    assert np.allclose(Qhat[0, 0], vals["Qhat_1"], atol=1e-12)
    assert np.allclose(Qhat[1, 0], vals["Qhat_2"], atol=1e-12)


def test_eq1_single_context_and_bias_off():
    Q_que = rng.normal(size=(4, 16))
    q_loc = rng.normal(size=(1, 4, 16))
    assert np.array_equal(O.personalized_query(Q_que, q_loc)[0], Q_que)
    q_loc5 = rng.normal(size=(5, 4, 16))
    out = O.personalized_query(Q_que, q_loc5, use_bias=False)
    assert out.shape == (5, 4, 16)
    for i in range(5):
        assert np.array_equal(out[i], Q_que)


def test_eq1_orthogonal_and_identical_local_queries():
    Q_que = np.zeros((1, 4)); Q_que[0, 0] = 2.0
    q_loc = np.zeros((3, 1, 4)); q_loc[:, 0, 1] = [1.0, -3.0, 5.0]       # all orthogonal to Q_que
    assert np.allclose(O.personalized_query(Q_que, q_loc), Q_que[None], atol=1e-15)
    Q_que = rng.normal(size=(2, 8))
    q_loc = np.repeat(Q_que[None], 4, axis=0)                            # cos = 1 for every j
    assert np.allclose(O.personalized_query(Q_que, q_loc), 2 * Q_que[None], atol=1e-12)


def test_eq1_excludes_own_document_and_normalises_by_D_minus_1():
    # D=3, orthonormal-ish construction where each document contributes a known amount
    Q_que = np.array([[1.0, 0.0, 0.0]])
    q_loc = np.array([[[1.0, 0.0, 0.0]],      # cos = 1
                      [[0.0, 2.0, 0.0]],      # cos = 0 -> contributes nothing
                      [[-3.0, 0.0, 0.0]]])    # cos = -1 -> |cos| = 1, vector keeps its sign
    Qhat = O.personalized_query(Q_que, q_loc)
    assert np.allclose(Qhat[0, 0], [1 + (0 + -3.0) / 2, 0, 0])
    assert np.allclose(Qhat[1, 0], [1 + (1.0 - 3.0) / 2, 0, 0])
    assert np.allclose(Qhat[2, 0], [1 + (1.0 + 0) / 2, 0, 0])


def test_eq1_sign_scale_and_permutation_properties():
    D, Hq, d = 4, 2, 8
    Q_que = rng.normal(size=(Hq, d))
    q_loc = rng.normal(size=(D, Hq, d))
    base = O.personalized_query(Q_que, q_loc)
    # flipping q_loc_j flips only term j (|cos| unchanged)
    flipped = q_loc.copy(); flipped[2] *= -1
    out = O.personalized_query(Q_que, flipped)
    for hq in range(Hq):
        w = abs(q_loc[2, hq] @ Q_que[hq]) / np.linalg.norm(q_loc[2, hq]) / np.linalg.norm(Q_que[hq])
        for i in (0, 1, 3):
            assert np.allclose(base[i, hq] - out[i, hq], 2 * w * q_loc[2, hq] / (D - 1), atol=1e-12)
        assert np.allclose(base[2, hq], out[2, hq], atol=1e-15)
    # scaling q_loc_j by a>0 scales term j by a
    scaled = q_loc.copy(); scaled[1] *= 3.0
    out = O.personalized_query(Q_que, scaled)
    assert np.allclose(out[0] - base[0], 2.0 * _term(Q_que, q_loc, 1) / (D - 1), atol=1e-12)
    assert np.allclose(out[1], base[1], atol=1e-15)                       # document 1 never sees its own term
    # permuting the contexts permutes Q^
    perm = [2, 0, 3, 1]
    out = O.personalized_query(Q_que, q_loc[perm])
    assert np.allclose(out, base[perm], atol=1e-12)
    # zero-norm local query: weight 0, no NaN
    z = q_loc.copy(); z[0] = 0
    assert np.isfinite(O.personalized_query(Q_que, z)).all()


def _term(Q_que, q_loc, j):
    out = np.zeros_like(Q_que)
    for hq in range(Q_que.shape[0]):
        w = abs(q_loc[j, hq] @ Q_que[hq]) / np.linalg.norm(q_loc[j, hq]) / np.linalg.norm(Q_que[hq])
        out[hq] = w * q_loc[j, hq]
    return out


def test_eq1_cos_is_per_head():
    # two heads with different cosines must get different weights
    Q_que = np.array([[1.0, 0.0], [1.0, 0.0]])
    q_loc = np.array([[[0.0, 0.0], [0.0, 0.0]], [[1.0, 0.0], [0.0, 1.0]]])
    Qhat = O.personalized_query(Q_que, q_loc)
    assert np.allclose(Qhat[0, 0], [2.0, 0.0]) and np.allclose(Qhat[0, 1], [1.0, 0.0])


def test_fold_gqa_group_mean_and_identity():
    Qhat = rng.normal(size=(3, 6, 4))
    assert np.array_equal(O.fold_gqa(Qhat, 6), Qhat)
    q = O.fold_gqa(Qhat, 2)
    assert np.allclose(q[:, 0], Qhat[:, 0:3].mean(axis=1)) and np.allclose(q[:, 1], Qhat[:, 3:6].mean(axis=1))


# ----------------------------------------------------------------------------- scores
def test_token_scores_against_matmul_and_context_routing():
    ctx = [0, 5, 12, 20]
    q = rng.normal(size=(3, 2, 8))
    K = rng.normal(size=(2, 20, 8))
    s = O.token_scores(q, K, ctx)
    for c in range(3):
        ref = torch.einsum("htd,hd->ht", torch.from_numpy(K[:, ctx[c]:ctx[c + 1]]), torch.from_numpy(q[c])).numpy()
        assert np.allclose(s[:, ctx[c]:ctx[c + 1]], ref, atol=1e-12)
    # context c uses q[c] only: changing q[1] leaves contexts 0 and 2 untouched
    q2 = q.copy(); q2[1] += 1.0
    s2 = O.token_scores(q2, K, ctx)
    assert np.array_equal(s2[:, :5], s[:, :5]) and np.array_equal(s2[:, 12:], s[:, 12:])
    assert not np.allclose(s2[:, 5:12], s[:, 5:12])


def test_unit_score_equals_score_of_mean_key():
    ctx = [0, 37, 101]                       # ragged: last units are short
    B = 8
    q = rng.normal(size=(2, 2, 16))
    K = rng.normal(size=(2, 101, 16))
    u = O.unit_scores(O.token_scores(q, K, ctx), ctx, B)
    nb, off = O.unit_layout(ctx, B)
    assert nb == [5, 8] and off == [0, 5, 13]
    for c in range(2):
        for m in range(nb[c]):
            a = ctx[c] + m * B
            b = min(a + B, ctx[c + 1])
            for h in range(2):
                assert abs(u[h, off[c] + m] - q[c, h] @ K[h, a:b].mean(axis=0)) < 1e-12
    # token mode: units are the tokens
    assert np.array_equal(O.unit_scores(O.token_scores(q, K, ctx), ctx, 1), O.token_scores(q, K, ctx))


# ----------------------------------------------------------------------------- selection
def test_protected_units_ranges():
    assert O.protected_units(256, 1, 4, 8) == list(range(4)) + list(range(248, 256))
    assert O.protected_units(1024, 64, 64, 128) == [0, 14, 15]
    assert O.protected_units(100, 16, 16, 32) == [0, 4, 5, 6]          # 100-32=68: units 4 (64..80),5,6(96..100)
    assert O.protected_units(10, 1, 8, 8) == list(range(10))           # overlap: everything protected
    assert O.protected_units(50, 1, 0, 0) == []


def test_budget_units():
    assert O.budget_units(256, 1, 4, 8, 1500) == 38
    assert O.budget_units(1024, 1, 16, 32, 1500) == 153
    assert O.budget_units(1536, 1, 16, 32, 1500) == 230
    assert O.budget_units(2048, 1, 16, 32, 1500) == 307
    assert O.budget_units(2048, 1, 16, 32, 500) == 102
    assert O.budget_units(2048, 1, 16, 32, 10000) == 2048
    assert O.budget_units(2048, 64, 64, 128, 500) == 3                  # clamped up to the protected count


def _brute_force_select(u_row, L_c, B, n_init, n_local, k):
    """Enumerate: the kept middle set is the size-(k-n_prot) subset that is lexicographically
    best under (score desc, index asc); found by repeatedly taking the best remaining unit."""
    nb = -(-L_c // B)
    prot = [m for m in range(nb) if m * B < n_init or min((m + 1) * B, L_c) > L_c - n_local]
    rest = [m for m in range(nb) if m not in prot]
    picked = []
    for _ in range(k - len(prot)):
        best = None
        for m in rest:
            if m in picked:
                continue
            if best is None or u_row[m] > u_row[best]:      # strict: first (lowest) index wins ties
                best = m
        picked.append(best)
    return sorted(prot + picked)


@pytest.mark.parametrize("seed", range(6))
def test_select_against_brute_force_with_ties(seed):
    r = np.random.default_rng(seed)
    lens = [int(x) for x in r.integers(20, 64, size=3)]
    ctx = [0] + list(np.cumsum(lens))
    B = [1, 1, 4, 8, 1, 2][seed]
    n_init, n_local = B * 1, B * 2
    nb, off = O.unit_layout(ctx, B)
    u = r.integers(0, 6, size=(2, off[-1])).astype(np.float64)         # many exact ties
    k_units = []
    for c in range(3):
        n_prot = len(O.protected_units(lens[c], B, n_init, n_local))
        k_units.append(int(r.integers(n_prot, nb[c] + 1)))
    sel = O.select_units(u, ctx, B, n_init, n_local, k_units)
    assert sel.shape == (2, sum(k_units))
    for h in range(2):
        pos = 0
        for c in range(3):
            exp = _brute_force_select(u[h, off[c]:off[c + 1]], lens[c], B, n_init, n_local, k_units[c])
            got = sel[h, pos:pos + k_units[c]] - off[c]
            assert list(got) == exp
            pos += k_units[c]
        assert np.all(np.diff(sel[h]) > 0)                               # strictly ascending


def test_select_edges_all_protected_only_monotone():
    ctx = [0, 40, 90]
    B, n_init, n_local = 1, 3, 5
    u = rng.normal(size=(1, 90))
    # k = nb -> everything
    sel = O.select_units(u, ctx, B, n_init, n_local, [40, 50])
    assert list(sel[0]) == list(range(90))
    # k = n_prot -> exactly the protected units (the paper's "no selection" ablation)
    sel = O.select_units(u, ctx, B, n_init, n_local, [8, 8])
    assert list(sel[0]) == [0, 1, 2, 35, 36, 37, 38, 39, 40, 41, 42, 85, 86, 87, 88, 89]
    # k -> k+1 adds exactly one index
    prev = set(O.select_units(u, ctx, B, n_init, n_local, [8, 8])[0])
    for k in range(9, 30):
        cur = set(O.select_units(u, ctx, B, n_init, n_local, [k, 8])[0])
        assert prev < cur and len(cur) == len(prev) + 1
        prev = cur
    # planted duplicate scores: the lower index is the one kept
    u2 = np.zeros((1, 90)); u2[0, 10] = 5.0; u2[0, 20] = 5.0
    sel = O.select_units(u2, ctx, B, n_init, n_local, [9, 8])
    assert 10 in sel[0] and 20 not in sel[0]
    # highest score wins over position
    u3 = np.zeros((1, 90)); u3[0, 30] = 1.0
    sel = O.select_units(u3, ctx, B, n_init, n_local, [9, 8])
    assert 30 in sel[0]


def test_kth_middle_score():
    ctx = [0, 20]
    u = np.arange(20, dtype=float)
    assert O.kth_middle_score(u, ctx, 1, 2, 2, [7], 0) == 15.0           # middle 2..17, keeps 17,16,15
    assert O.kth_middle_score(u, ctx, 1, 2, 2, [4], 0) is None


# ----------------------------------------------------------------------------- compaction
def test_compact_is_exact_gather_and_inverse_map_round_trips():
    ctx = [0, 30, 75]
    B = 4
    K = rng.normal(size=(2, 75, 8)).astype(np.float32)
    V = rng.normal(size=(2, 75, 8)).astype(np.float32)
    nb, off = O.unit_layout(ctx, B)                                      # nb = [8, 12]; unit 7 of ctx0 is short (2 tokens)
    u = rng.normal(size=(2, off[-1]))
    sel = O.select_units(u, ctx, B, 4, 4, [4, 5])
    Kc, Vc, S, inv = O.compact(K, V, sel, ctx, B)
    assert S == (4 * 4 - 2) + (5 * 4 - 3)                                # short tails of both contexts are protected
    for h in range(2):
        toks = O.units_to_tokens(sel[h], ctx, B)
        assert np.all(np.diff(toks) > 0)
        assert np.array_equal(Kc[h, :S], K[h, toks]) and np.array_equal(Vc[h, :S], V[h, toks])
        assert np.array_equal(inv[h, toks], np.arange(S))
        assert (inv[h] >= 0).sum() == S
    # 100 %: the compact cache is the concatenation itself
    sel = O.select_units(u, ctx, B, 4, 4, nb)
    Kc, Vc, S, inv = O.compact(K, V, sel, ctx, B, capacity=80)
    assert S == 75 and np.array_equal(Kc[:, :75], K) and np.array_equal(Vc[:, :75], V) and Kc.shape[1] == 80
    assert np.array_equal(inv, np.tile(np.arange(75), (2, 1)))


# ----------------------------------------------------------------------------- update
def test_round_to_bf16_matches_torch():
    x = rng.normal(size=4096) * np.exp(rng.normal(size=4096) * 4)
    x = np.concatenate([x, [1.00390625, 1.01171875, -1.00390625, 0.0, 3.0]])   # exact ties to even
    ref = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).double().numpy()
    assert np.array_equal(O.round_to_bf16(x), ref)


def test_fusion_closed_forms():
    old = rng.normal(size=16)
    assert np.allclose(O.fuse_row(old.copy(), old), old, atol=1e-14)                 # new = old
    assert np.allclose(O.fuse_row(2.5 * old, old), 2.5 * old, atol=1e-14)            # theta = 1 -> new
    orth = rng.normal(size=16); orth -= (orth @ old) / (old @ old) * old
    assert np.allclose(O.fuse_row(orth, old), old, atol=1e-12)                       # theta = 0 -> old
    assert np.allclose(O.fuse_row(-old, old), 3 * old, atol=1e-14)                   # theta = -1 -> -(-old)+2 old
    assert np.allclose(O.fuse_row(np.zeros(16), old), np.zeros(16))                  # zero norm: replaced
    # generic: weights sum to one => fusing along the segment keeps affine combinations
    new = rng.normal(size=16)
    th = (new @ old) / np.linalg.norm(new) / np.linalg.norm(old)
    out = O.fuse_row(new, old)
    assert np.allclose(out - old, th * (new - old), atol=1e-14)


def test_update_overwrite_fusion_skip_rules():
    Hkv, cap, d, L_tot = 2, 6, 4, 10
    Kc = rng.normal(size=(Hkv, cap, d)); Vc = rng.normal(size=(Hkv, cap, d))
    inv = np.full((Hkv, L_tot), -1, dtype=np.int32)
    inv[0, [1, 4, 7]] = [0, 1, 2]
    inv[1, [1, 5, 7]] = [0, 1, 2]
    tok = [4, -1, 7, 9]                       # 4: only head 0 kept it; -1: skip; 7: both; 9: nobody
    Kn = rng.normal(size=(4, Hkv, d)); Vn = rng.normal(size=(4, Hkv, d))
    K2, V2 = O.update(Kc, Vc, inv, tok, Kn, Vn, "overwrite")
    assert np.array_equal(K2[0, 1], Kn[0, 0]) and np.array_equal(V2[0, 1], Vn[0, 0])
    assert np.array_equal(K2[0, 2], Kn[2, 0]) and np.array_equal(K2[1, 2], Kn[2, 1])
    mask = np.ones((Hkv, cap), bool); mask[0, 1] = mask[0, 2] = mask[1, 2] = False
    assert np.array_equal(K2[mask], Kc[mask]) and np.array_equal(V2[mask], Vc[mask])  # untouched slots identical
    K3, V3 = O.update(Kc, Vc, inv, tok, Kn, Vn, "fusion")
    assert np.allclose(K3[1, 2], O.fuse_row(Kn[2, 1], Kc[1, 2])) and np.allclose(V3[0, 1], O.fuse_row(Vn[0, 0], Vc[0, 1]))
    assert np.array_equal(K3[mask], Kc[mask])
    # K and V use their own theta
    assert not np.allclose((K3[0, 1] - Kc[0, 1]) / (Kn[0, 0] - Kc[0, 1]), (V3[0, 1] - Vc[0, 1]) / (Vn[0, 0] - Vc[0, 1]))
    # bf16 rounding of the fused row
    K4, _ = O.update(Kc, Vc, inv, tok, Kn, Vn, "fusion", dtype="bf16")
    assert np.array_equal(K4[0, 1], O.round_to_bf16(K3[0, 1]))


# ----------------------------------------------------------------------------- attention
def _sdpa_ref(Kc, Vc, cache_len, Q, Kq, Vq, scale=None):
    """Independent library route: torch fp64 scaled_dot_product_attention with heads repeated
    G times and an explicit boolean mask."""
    T_q, Hq, d = Q.shape
    Hkv = Kc.shape[0]
    G = Hq // Hkv
    K = torch.from_numpy(Kc[:, :cache_len]).double()
    V = torch.from_numpy(Vc[:, :cache_len]).double()
    n_app = 0
    if Kq is not None:
        K = torch.cat([K, torch.from_numpy(Kq).double().permute(1, 0, 2)], dim=1)
        V = torch.cat([V, torch.from_numpy(Vq).double().permute(1, 0, 2)], dim=1)
        n_app = T_q
    S = K.shape[1]
    mask = torch.ones(T_q, S, dtype=torch.bool)
    for t in range(T_q):
        for j in range(n_app):
            if j > t:
                mask[t, cache_len + j] = False
    q = torch.from_numpy(Q).double().permute(1, 0, 2)[None]             # [1, Hq, T, d]
    k = K.repeat_interleave(G, dim=0)[None]
    v = V.repeat_interleave(G, dim=0)[None]
    out = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask[None, None], scale=scale)
    return out[0].permute(1, 0, 2).numpy()


def test_attention_against_torch_sdpa():
    Hkv, Hq, d, cap, S, T = 2, 6, 8, 40, 29, 5
    Kc = rng.normal(size=(Hkv, cap, d)); Vc = rng.normal(size=(Hkv, cap, d))
    Q = rng.normal(size=(T, Hq, d)); Kq = rng.normal(size=(T, Hkv, d)); Vq = rng.normal(size=(T, Hkv, d))
    out, lse, K2, V2, n = O.attention(Kc, Vc, S, Q, Kq, Vq)
    assert n == S + T
    assert np.allclose(out, _sdpa_ref(Kc, Vc, S, Q, Kq, Vq), atol=1e-12)
    assert np.array_equal(K2[:, S:S + T], Kq.transpose(1, 0, 2)) and np.array_equal(V2[:, S:S + T], Vq.transpose(1, 0, 2))
    assert np.array_equal(K2[:, :S], Kc[:, :S])
    out2, _, _, _, n2 = O.attention(Kc, Vc, S, Q, None, None, scale=0.3)
    assert n2 == S and np.allclose(out2, _sdpa_ref(Kc, Vc, S, Q, None, None, scale=0.3), atol=1e-12)


def test_attention_softmax_invariants():
    Hkv, Hq, d, S, T = 1, 2, 4, 9, 3
    Kc = rng.normal(size=(Hkv, S, d)); Vc = rng.normal(size=(Hkv, S, d)); Q = rng.normal(size=(T, Hq, d))
    # rows sum to one: with V = ones the output is ones
    out, lse, *_ = O.attention(Kc, np.ones_like(Vc), S, Q)
    assert np.allclose(out, 1.0, atol=1e-14)
    # lse is the log of the softmax denominator
    for t in range(T):
        for hq in range(Hq):
            assert abs(lse[hq, t] - math.log(sum(math.exp(0.5 * float(Kc[0, s] @ Q[t, hq])) for s in range(S)))) < 1e-12
    # one visible slot => that V row
    out, *_ = O.attention(Kc, Vc, 1, Q)
    assert np.allclose(out, Vc[0, 0][None, None], atol=1e-14)
    # all keys equal => mean of V
    out, *_ = O.attention(np.repeat(Kc[:, :1], S, 1), Vc, S, Q)
    assert np.allclose(out, Vc[0].mean(0)[None, None], atol=1e-13)
    # all V rows equal => that row
    out, *_ = O.attention(Kc, np.repeat(Vc[:, :1], S, 1), S, Q)
    assert np.allclose(out, Vc[0, 0][None, None], atol=1e-13)
    # joint permutation of cache slots changes nothing
    p = rng.permutation(S)
    a, *_ = O.attention(Kc, Vc, S, Q)
    b, *_ = O.attention(Kc[:, p], Vc[:, p], S, Q)
    assert np.allclose(a, b, atol=1e-13)
    # slots beyond cache_len are invisible
    Kj = np.concatenate([Kc, 100 * np.ones((1, 3, d))], 1); Vj = np.concatenate([Vc, 1e6 * np.ones((1, 3, d))], 1)
    c, *_ = O.attention(Kj, Vj, S, Q)
    assert np.allclose(a, c, atol=1e-13)


def test_attention_causal_tail_first_token_sees_only_itself_of_the_chunk():
    Hkv, Hq, d, T = 1, 1, 4, 3
    Kc = np.zeros((1, 3, d)); Vc = np.zeros((1, 3, d))
    Q = rng.normal(size=(T, Hq, d)); Kq = rng.normal(size=(T, Hkv, d)); Vq = rng.normal(size=(T, Hkv, d))
    out, *_ = O.attention(Kc, Vc, 0, Q, Kq, Vq)
    assert np.allclose(out[0, 0], Vq[0, 0], atol=1e-14)                   # token 0 sees only appended slot 0
    # last token sees all three
    lg = 0.5 * (Kq[:, 0] @ Q[2, 0]); p = np.exp(lg - lg.max()); p /= p.sum()
    assert np.allclose(out[2, 0], p @ Vq[:, 0], atol=1e-13)


def test_attention_split_merge_identity():
    """Merging two halves via (max, sum) statistics equals the one-shot result: the identity
    every split-KV kernel relies on, checked on the oracle's lse output."""
    Hkv, Hq, d, S, T = 1, 2, 8, 32, 2
    Kc = rng.normal(size=(Hkv, S, d)); Vc = rng.normal(size=(Hkv, S, d)); Q = rng.normal(size=(T, Hq, d))
    full, lse, *_ = O.attention(Kc, Vc, S, Q)
    o1, l1, *_ = O.attention(Kc[:, :13], Vc[:, :13], 13, Q)
    o2, l2, *_ = O.attention(Kc[:, 13:], Vc[:, 13:], S - 13, Q)
    for t in range(T):
        for hq in range(Hq):
            m = max(l1[hq, t], l2[hq, t])
            w1, w2 = math.exp(l1[hq, t] - m), math.exp(l2[hq, t] - m)
            merged = (w1 * o1[t, hq] + w2 * o2[t, hq]) / (w1 + w2)
            assert np.allclose(merged, full[t, hq], atol=1e-13)
            assert abs(m + math.log(w1 + w2) - lse[hq, t]) < 1e-12


# ----------------------------------------------------------------------------- end to end
def _tiny_problem(seed=3, D=3, L_c=24, Hq=4, Hkv=2, d=8, T_q=4, T_loc=3):
    r = np.random.default_rng(seed)
    ctx = [L_c * i for i in range(D + 1)]
    K = r.normal(size=(Hkv, D * L_c, d)); V = r.normal(size=(Hkv, D * L_c, d))
    Q = r.normal(size=(T_q, Hq, d)); Qloc = r.normal(size=(D, T_loc, Hq, d))
    return ctx, K, V, Q, Qloc, r


def test_full_budget_equals_full_attention_over_concatenation():
    ctx, K, V, Q, Qloc, r = _tiny_problem()
    res = O.sparsify(K, V, Q, Qloc, ctx, 1, 2, 3, [24, 24, 24])
    Qa = r.normal(size=Q.shape)
    out, *_ = O.attention(res["Kc"], res["Vc"], res["cache_len"], Qa)
    ref = _sdpa_ref(K, V, K.shape[1], Qa, None, None)
    assert res["cache_len"] == 72 and np.allclose(out, ref, atol=1e-12)


def test_consensus_probe_bias_reaches_selection():
    """Plant, in context 0, one middle key aligned with context 1's local query and orthogonal
    to the pooled user query: with the Eq. 1 bias it is kept, without the bias it is not."""
    ctx, K, V, Q, Qloc, r = _tiny_problem(D=2, Hq=2, Hkv=2, L_c=40)
    Q_que = O.pool_query(Q); q_loc = O.pool_local(Qloc)
    K = K * 0.05
    for h in range(2):
        v = q_loc[1, h] - (q_loc[1, h] @ Q_que[h]) / (Q_que[h] @ Q_que[h]) * Q_que[h]
        K[h, 17] = 10.0 * v / np.linalg.norm(v)
    k_units = [6, 6]                                                      # 5 protected + 1 free pick
    with_bias = O.sparsify(K, V, Q, Qloc, ctx, 1, 2, 3, k_units, use_bias=True)
    without = O.sparsify(K, V, Q, Qloc, ctx, 1, 2, 3, k_units, use_bias=False)
    assert all(17 in with_bias["sel"][h] for h in range(2))
    assert abs(without["s"][0, 17]) < 1e-9                                # orthogonal to Q_que: score exactly ~0
    # and the personalised queries of the two contexts differ (each leaves out its own document)
    assert not np.allclose(with_bias["Qhat"][0], with_bias["Qhat"][1])


def test_sparsify_stage_shapes_and_counts():
    ctx, K, V, Q, Qloc, r = _tiny_problem()
    res = O.sparsify(K, V, Q, Qloc, ctx, 4, 4, 4, [3, 4, 2])
    assert res["sel"].shape == (2, 9) and res["cache_len"] == 36
    assert res["u"].shape == (2, 18) and res["s"].shape == (2, 72)
    nb, off = O.unit_layout(ctx, 4)
    for h in range(2):
        counts = [int(((res["sel"][h] >= off[c]) & (res["sel"][h] < off[c + 1])).sum()) for c in range(3)]
        assert counts == [3, 4, 2]


# ----------------------------------------------------------------------------- Eq. 2 / Eq. 3 / cross-context Top-K
def test_eq2_hand_values_and_interval_ends():
    assert O.top_p_ratio(s_anc=2.0, s_max=4.0, s_min=0.0) == 0.5
    assert O.top_p_ratio(1.0, 4.0, 0.0) == 0.75                       # a low anchor lets more blocks through
    assert O.top_p_ratio(4.0, 4.0, 0.0) == 0.0                        # s_anc = s_max: inside the interval, P = 0
    assert O.top_p_ratio(0.0, 4.0, 0.0) == 0.0                        # s_anc = s_min: outside (open end)
    assert O.top_p_ratio(5.0, 4.0, 0.0) == 0.0 and O.top_p_ratio(-1.0, 4.0, 0.0) == 0.0
    assert O.top_p_ratio(1.0, 1.0, 1.0) == 0.0                        # degenerate: no division by zero
    assert abs(O.top_p_ratio(1e-9, 1.0, 0.0) - 1.0) < 1e-8            # s_anc -> s_min+ : P -> 1


def test_anchor_score_is_token_weighted_mean_of_protected_units():
    ctx = [0, 22]                     # B = 4: units of 4,4,4,4,4,2 tokens; init = unit 0, local (last 4 tokens) = units 4,5
    u = np.array([10.0, 1.0, 2.0, 3.0, 20.0, 40.0])
    assert O.protected_units(22, 4, 4, 4) == [0, 4, 5]
    assert O.anchor_score(u, 0, ctx, 4, 4, 4) == pytest.approx((10 * 4 + 20 * 4 + 40 * 2) / 10)
    assert O.middle_units(22, 4, 4, 4) == [1, 2, 3]


def test_top_p_per_head_default_and_caller_blocks_and_eq3():
    ctx = [0, 24, 40]                 # B = 4, init 4, local 4 -> ctx0 units 0..5 (middle 1..4), ctx1 units 6..9 (middle 7,8)
    u = np.array([[2.0, 5.0, 1.0, 3.0, 4.0, 2.0,   0.0, 9.0, 1.0, 0.0],
                  [9.0, 5.0, 1.0, 3.0, 4.0, 9.0,   3.0, 2.0, 6.0, 3.0]])
    P = O.top_p_per_head(u, ctx, 4, 4, 4)
    # head 0 ctx 0: anc = 2, max 5, min 1 -> 3/4 ; ctx 1: anc 0 < min 1 -> 0
    # head 1 ctx 0: anc 9 > max -> 0 ;           ctx 1: anc 3, max 6, min 2 -> 3/4
    assert np.allclose(P, [[0.75, 0.0], [0.0, 0.75]])
    P2 = O.top_p_per_head(u, ctx, 4, 4, 4, max_units=[4, 8], min_units=[3, 7])   # caller-supplied max/min blocks
    # head 0 ctx 0: max 4, min 3, anc 2 -> not in (3,4] -> 0 ; ctx 1: max 1, min 9 -> empty interval -> 0
    # head 1 ctx 0: 0 ; ctx 1: max 6, min 2, anc 3 -> 0.75
    assert np.allclose(P2, [[0.0, 0.0], [0.0, 0.75]])
    Pd = O.consolidate_top_p(np.stack([P, P2]))                      # Eq. 3 over two "stable layers" (and the heads)
    assert np.allclose(Pd, [0.75 / 4, (0.75 + 0.75) / 4])
    assert O.candidate_counts([0.74, 0.5, 1.0, 0.0], [0, 24, 40, 64, 88], 4, 4, 4) == [2, 1, 4, 0]


def _cross_brute(u_row, ctx, B, n_init, n_local, cand):
    """Independent route with numpy argsort on a (score, id) structured key."""
    nb, off = O.unit_layout(ctx, B)
    D = len(nb)
    pool_v, pool_id, prot = [], [], []
    for c in range(D):
        L_c = ctx[c + 1] - ctx[c]
        pr = O.protected_units(L_c, B, n_init, n_local)
        prot += [off[c] + m for m in pr]
        mid = np.array([m for m in range(nb[c]) if m not in set(pr)], dtype=int)
        if len(mid) == 0 or cand[c] == 0:
            continue
        vals = u_row[off[c] + mid]
        order = np.lexsort((mid, -vals))[: cand[c]]
        lo, hi = vals.min(), vals.max()
        pool_v += list(((vals[order] - lo) / (hi - lo)) if hi > lo else np.zeros(len(order)))
        pool_id += list(off[c] + mid[order])
    K = sum(cand) // D
    pool_v, pool_id = np.array(pool_v), np.array(pool_id, dtype=int)
    pick = np.lexsort((pool_id, -pool_v))[:K] if len(pool_v) else []
    return sorted(prot + [int(pool_id[i]) for i in pick])


@pytest.mark.parametrize("seed", range(5))
def test_cross_context_select_against_brute_force(seed):
    r = np.random.default_rng(100 + seed)
    B = [1, 4, 8, 2, 1][seed]
    lens = [int(x) for x in r.integers(6 * B, 20 * B, size=4)]
    ctx = [0] + [int(x) for x in np.cumsum(lens)]
    nb, off = O.unit_layout(ctx, B)
    u = r.integers(0, 7, size=(2, off[-1])).astype(float) if seed % 2 else r.normal(size=(2, off[-1]))
    cand = [int(r.integers(0, len(O.middle_units(lens[c], B, B, 2 * B)) + 1)) for c in range(4)]
    sel, counts = O.cross_context_select(u, ctx, B, B, 2 * B, cand)
    K = sum(cand) // 4
    n_prot = sum(len(O.protected_units(n, B, B, 2 * B)) for n in lens)
    assert sel.shape == (2, n_prot + K)
    for h in range(2):
        assert list(sel[h]) == _cross_brute(u[h], ctx, B, B, 2 * B, cand)
        assert counts[h].sum() == n_prot + K and np.all(np.diff(sel[h]) > 0)


def test_cross_context_select_properties():
    r = np.random.default_rng(7)
    ctx = [0, 30, 70, 95]
    u = r.normal(size=(1, 95))
    cand = [6, 9, 4]
    sel, counts = O.cross_context_select(u, ctx, 1, 2, 3, cand)
    # min-max normalisation: an affine map (a > 0) of one context's scores changes nothing
    u2 = u.copy(); u2[0, 30:70] = 3.5 * u2[0, 30:70] - 11.0
    sel2, _ = O.cross_context_select(u2, ctx, 1, 2, 3, cand)
    assert np.array_equal(sel, sel2)
    # one context: K = all its candidates, i.e. the fixed-budget selection with k = protected + candidates
    s1, c1 = O.cross_context_select(u[:, :30], [0, 30], 1, 2, 3, [6])
    assert np.array_equal(s1, O.select_units(u[:, :30], [0, 30], 1, 2, 3, [5 + 6]))
    # nothing retrieved: only the protected units survive (the "no selection" ablation)
    s0, c0 = O.cross_context_select(u, ctx, 1, 2, 3, [0, 0, 0])
    assert list(s0[0]) == [0, 1, 27, 28, 29, 30, 31, 67, 68, 69, 70, 71, 92, 93, 94]
    # the best unit of a context normalises to 1 and always wins a place when K >= number of contexts with candidates
    for c in range(3):
        lo, hi = ctx[c] + 2, ctx[c + 1] - 3
        assert (lo + int(np.argmax(u[0, lo:hi]))) in sel[0]


# ------------------------------------------------------------------------------------------
# Section 3.3: blank-block alignment and the two recomputation rules
# ------------------------------------------------------------------------------------------
def test_align_layers_the_four_cases_of_the_recomputation_figure():
    """tests/golden/recompute_figure_cases.txt: the four token cases of the paper's recomputation figure (plus two
    corner tokens) as a two-layer, one-head example with the flags the text prescribes for each."""
    letters = {"K": O.FLAG_KEPT, "R": O.FLAG_RECOMPUTE, "O": O.FLAG_OUTPUT, "P": O.FLAG_PAD_REUSE}
    rows = []
    with open(os.path.join(GOLDEN, "recompute_figure_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            body = line.split("=")[1]
            bits, lower, upper = [x.strip() for x in body.split("|")]
            rows.append(([int(x) for x in bits.split(",")], lower, upper))
    T = len(rows)
    assert T == 6
    inv = np.full((2, 1, T), -1, dtype=np.int32)
    lists = [[], []]
    for t, (bits, _, _) in enumerate(rows):
        for n in range(2):
            if bits[n]:
                inv[n, 0, t] = int((inv[n, 0, :t] >= 0).sum())          # slots in token order
            if bits[2 + n]:
                lists[n].append(t)
    R = max(len(x) for x in lists) + 1
    tok = np.array([x + [-1] * (R - len(x)) for x in lists])
    flags, merged, run = O.align_layers(inv, tok)
    for t, (_, lower, upper) in enumerate(rows):
        for n, want in enumerate((lower, upper)):
            expect = sum(letters[ch] for ch in want if ch in letters)
            assert flags[n, t] == expect, f"token {t + 1} layer {n}: {flags[n, t]} != {want}"
    assert merged.tolist() == [0, 1, 2, 3, 5]                              # token 5 is kept by no layer
    assert run[0].tolist() == [0, 2, 3, 5] and run[1].tolist() == [2, 3, 5]


@pytest.mark.parametrize("seed", range(5))
def test_align_layers_plan_is_sufficient_and_minimal(seed):
    """Demand analysis written the other way round: the hidden state of t is needed at the input of layer n iff
    layer n recomputes t or the input of layer n+1 needs it.  The plan's forward lists must be exactly these
    sets, and each layer's outputs exactly the next layer's inputs."""
    r = np.random.default_rng(seed)
    L, Hkv, T, R = int(r.integers(1, 7)), int(r.integers(1, 4)), 60, 9
    inv = np.where(r.random((L, Hkv, T)) < 0.35, 1, -1).astype(np.int32)
    tok = np.stack([r.permutation(T)[:R] for _ in range(L)])
    tok[r.random(tok.shape) < 0.2] = -1
    flags, merged, run = O.align_layers(inv, tok)
    kept = (inv >= 0).any(axis=1)                                            # [L, T]
    need = [set() for _ in range(L + 1)]
    for n in reversed(range(L)):
        rec_n = {int(t) for t in tok[n] if t >= 0 and kept[n, t]}
        need[n] = rec_n | need[n + 1]
        assert {t for t in range(T) if flags[n, t] & O.FLAG_RECOMPUTE} == rec_n
    for n in range(L):
        assert set(run[n].tolist()) == need[n]
        assert {t for t in range(T) if flags[n, t] & O.FLAG_OUTPUT} == need[n + 1]
        assert np.all(np.diff(run[n]) > 0)
    assert not (flags[L - 1] & O.FLAG_OUTPUT).any()
    assert merged.tolist() == [t for t in range(T) if kept[:, t].any()]
    pad = (flags & O.FLAG_PAD_REUSE) != 0
    assert np.array_equal(pad, ((flags & O.FLAG_OUTPUT) != 0) & ~kept & ((flags & O.FLAG_RECOMPUTE) == 0))
    assert np.array_equal((flags & O.FLAG_KEPT) != 0, kept)


def test_align_layers_without_recomputation_only_marks_kept_tokens():
    inv = np.full((3, 2, 10), -1, dtype=np.int32)
    inv[0, 0, 2] = 0
    inv[2, 1, 7] = 0                                       # kept by one head only still counts as kept
    flags, merged, run = O.align_layers(inv, np.full((3, 4), -1))
    assert flags.sum() == 2 and flags[0, 2] == O.FLAG_KEPT and flags[2, 7] == O.FLAG_KEPT
    assert merged.tolist() == [2, 7] and all(len(x) == 0 for x in run)


# ------------------------------------------------------------------------------------------
# Section 3.2: blocks represented by the mean vector of their token caches
# ------------------------------------------------------------------------------------------
def test_block_means_hand_values_tail_and_token_mode():
    K = np.zeros((1, 5, 2))
    K[0] = [[1, 2], [3, 6], [10, 20], [30, 40], [7, 9]]
    off = [0, 2, 5]                                              # contexts of 2 and 3 tokens
    Kb = O.block_means(K, off, 2)
    assert Kb.shape == (1, 3, 2)
    assert Kb[0].tolist() == [[2, 4], [20, 30], [7, 9]]          # the short tail unit is its single token
    assert np.array_equal(O.block_means(K, off, 1), K)           # token mode: the representative is the key itself
    Kb4 = O.block_means(K, off, 4)                               # units never cross a context boundary
    assert Kb4[0].tolist() == [[2, 4], [47 / 3, 23]]


@pytest.mark.parametrize("B", [2, 8, 64])
def test_score_on_block_means_equals_block_mean_of_token_scores(B):
    """<q, mean_t K_t> = mean_t <q, K_t>: scoring the representatives reproduces the unit scores."""
    r = np.random.default_rng(B)
    lens = [130, 64, 7, 200]
    off = [0] + list(np.cumsum(lens))
    Hkv, d = 2, 16
    K = r.normal(size=(Hkv, off[-1], d))
    q = r.normal(size=(len(lens), Hkv, d))
    u_tok = O.unit_scores(O.token_scores(q, K, off), off, B)
    nb, unit_off = O.unit_layout(off, B)
    u_rep = O.token_scores(q, O.block_means(K, off, B), unit_off)
    assert np.allclose(u_tok, u_rep, rtol=0, atol=1e-12)


def test_block_means_rounding_to_storage_type():
    r = np.random.default_rng(5)
    K = O.round_to_bf16(r.normal(size=(1, 64, 8)))
    exact = O.block_means(K, [0, 64], 16)
    stored = O.block_means(K, [0, 64], 16, "bf16")
    assert np.array_equal(stored, O.round_to_bf16(stored))                     # representable
    assert (np.abs(stored - exact) <= 2.0 ** -8 * np.abs(exact)).all()   # half a bf16 ulp: 8 significant bits
    assert np.array_equal(O.block_means(K, [0, 64], 16, "f32"), exact.astype(np.float32).astype(np.float64))

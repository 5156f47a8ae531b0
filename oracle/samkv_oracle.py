"""SamKV hot-path oracle: a plain, slow CPU implementation in float64.

THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be checked
against something written directly from the paper ("Sparse Attention across
Multiple-context KV Cache").  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import it; the product path never does, and it shares no code
with the CUDA sources.

Every function works on ONE (layer, batch element) problem and on numpy float64
arrays (callers up-convert stored bf16 / fp32 values exactly; nothing is re-rounded
on the way in).  Loops over contexts, heads and tokens are written out; the only
library primitives used are `@` (matrix product), `np.sort`/`np.lexsort`, `np.exp`,
`np.log`.  There is no blocking, fusion or reordering.

Notation (paper, Table 2):  D contexts ("documents"), Q_que generic query vector,
Q_doc-j_loc local Q cache of document j, Q^_doc-i personalised query of document i,
<.,.> inner product.  Added here: Hq query heads, Hkv key/value heads, G = Hq/Hkv,
d head dimension, B selection-unit ("block") size in tokens, ctx_offsets[c] start of
context c on the concatenated token axis, k_units[c] units kept in context c.

Pins (tests/test_oracle_pins.py): closed forms of Eq. 1 and Eq. 4, linearity of the
block-mean score, brute-force selection, bit-exact gather, softmax invariants, the
100 %-budget == full-attention invariant, torch's fp64 scaled_dot_product_attention, hand
values / brute force / invariances for Eq. 2-3 and the cross-context Top-K, and for the
cross-layer alignment the four token cases of the paper's recomputation figure plus a
layer-by-layer simulation that checks the plan is sufficient and minimal.
The paper prints no worked numerical example of Eq. 1-4, so parity with the paper's
own numbers is unpinned; every function below is pinned by mathematics instead.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------------------
# Section 3.1 "Generate generic query vector": mean pooling over the sequence dimension
# --------------------------------------------------------------------------------------
def pool_query(Q: np.ndarray) -> np.ndarray:
    """Q_que[hq, :] = (1/T_q) sum_t Q[t, hq, :].   Q: [T_q, Hq, d] -> [Hq, d].

    Section 3.1: the user query's Q matrix of a layer is turned into one vector
    by mean pooling (arithmetic mean over the query tokens, per head).
    """
    Q = np.asarray(Q, dtype=F64)
    T_q = Q.shape[0]
    acc = np.zeros(Q.shape[1:], dtype=F64)
    for t in range(T_q):
        acc += Q[t]
    return acc / T_q


def pool_local(Qloc: np.ndarray) -> np.ndarray:
    """q_loc[j, hq, :] = (1/T_loc) sum_t Qloc[j, t, hq, :].   [D, T_loc, Hq, d] -> [D, Hq, d].

    Section 3.1 "Add personalized bias": document j's local Q cache enters Eq. 1
    as a vector; this build reads that as the mean over its local-position rows.
    """
    Qloc = np.asarray(Qloc, dtype=F64)
    D = Qloc.shape[0]
    out = np.zeros((D,) + Qloc.shape[2:], dtype=F64)
    for j in range(D):
        out[j] = pool_query(Qloc[j])
    return out


def _cos(a: np.ndarray, b: np.ndarray) -> float:
    na = np.sqrt(a @ a)
    nb = np.sqrt(b @ b)
    if na == 0.0 or nb == 0.0:
        return None
    return float((a @ b) / (na * nb))


# --------------------------------------------------------------------------------------
# Eq. 1: personalised query vector
# --------------------------------------------------------------------------------------
def personalized_query(Q_que: np.ndarray, q_loc: np.ndarray | None, use_bias: bool = True) -> np.ndarray:
    """Eq. 1, per query head:

        Q^_doc-i = Q_que + 1/(D-1) * sum_{j != i} |cos(Q_que, Q_doc-j_loc)| * Q_doc-j_loc

    Q_que: [Hq, d], q_loc: [D, Hq, d] -> Q^: [D, Hq, d].
    D == 1 (nothing to sum over) or use_bias False gives Q^ = Q_que (Section 2.1:
    with a single context the method reduces to the single-context case).
    A zero-norm operand of cos gives weight 0.
    """
    Q_que = np.asarray(Q_que, dtype=F64)
    Hq, d = Q_que.shape
    if q_loc is None or not use_bias:
        D = 1 if q_loc is None else q_loc.shape[0]
        return np.repeat(Q_que[None], D, axis=0).copy()
    q_loc = np.asarray(q_loc, dtype=F64)
    D = q_loc.shape[0]
    Qhat = np.zeros((D, Hq, d), dtype=F64)
    for i in range(D):
        for hq in range(Hq):
            bias = np.zeros(d, dtype=F64)
            if D > 1:
                for j in range(D):
                    if j == i:
                        continue
                    c = _cos(Q_que[hq], q_loc[j, hq])
                    w = 0.0 if c is None else abs(c)
                    bias += w * q_loc[j, hq]
                bias /= (D - 1)
            Qhat[i, hq] = Q_que[hq] + bias
    return Qhat


def fold_gqa(Qhat: np.ndarray, Hkv: int) -> np.ndarray:
    """q[i, h, :] = (1/G) sum_{g<G} Q^[i, h*G+g, :].   [D, Hq, d] -> [D, Hkv, d].

    The paper does not say how Hq personalised queries meet Hkv key heads under
    grouped-query attention; this build averages the G query heads of a group.
    """
    Qhat = np.asarray(Qhat, dtype=F64)
    D, Hq, d = Qhat.shape
    G = Hq // Hkv
    assert G * Hkv == Hq
    q = np.zeros((D, Hkv, d), dtype=F64)
    for i in range(D):
        for h in range(Hkv):
            for g in range(G):
                q[i, h] += Qhat[i, h * G + g]
            q[i, h] /= G
    return q


# --------------------------------------------------------------------------------------
# Section 3.2: inner-product scores, block = mean of its tokens
# --------------------------------------------------------------------------------------
def token_scores(q: np.ndarray, K: np.ndarray, ctx_offsets) -> np.ndarray:
    """s[h, t] = < q[c(t), h, :], K[h, t, :] >  (raw inner product, no scaling).

    q: [D, Hkv, d], K: [Hkv, L_tot, d] -> [Hkv, L_tot].  Section 3.2 scores the
    K cache of document i with that document's own Q^_doc-i.
    """
    q = np.asarray(q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    Hkv, L_tot, d = K.shape
    D = len(ctx_offsets) - 1
    s = np.zeros((Hkv, L_tot), dtype=F64)
    for c in range(D):
        lo, hi = int(ctx_offsets[c]), int(ctx_offsets[c + 1])
        for h in range(Hkv):
            s[h, lo:hi] = K[h, lo:hi, :] @ q[c, h]
    return s


def unit_layout(ctx_offsets, B: int):
    """Units ("blocks") of B tokens counted from each context's own start; the last
    unit of a context may be short.  Returns (nb[c], unit_off[c] (D+1 entries))."""
    D = len(ctx_offsets) - 1
    nb = [(-(-(int(ctx_offsets[c + 1]) - int(ctx_offsets[c])) // B)) for c in range(D)]
    unit_off = [0]
    for c in range(D):
        unit_off.append(unit_off[-1] + nb[c])
    return nb, unit_off


def unit_scores(s: np.ndarray, ctx_offsets, B: int) -> np.ndarray:
    """u[h, m] = mean of s[h, t] over the real tokens of unit m.  [Hkv, L_tot] -> [Hkv, U_tot].

    Section 3.2: a block is represented by the mean vector of its tokens' K; by
    linearity <q, mean K> equals the mean of the token scores, which is what is computed.
    """
    s = np.asarray(s, dtype=F64)
    Hkv = s.shape[0]
    nb, unit_off = unit_layout(ctx_offsets, B)
    u = np.zeros((Hkv, unit_off[-1]), dtype=F64)
    for c in range(len(nb)):
        lo, hi = int(ctx_offsets[c]), int(ctx_offsets[c + 1])
        for m in range(nb[c]):
            a = lo + m * B
            b = min(a + B, hi)
            for h in range(Hkv):
                u[h, unit_off[c] + m] = s[h, a:b].sum() / (b - a)
    return u


# --------------------------------------------------------------------------------------
# Section 3.2 / Section 4.1: protected initial + local blocks, top-k of the middle
# --------------------------------------------------------------------------------------
def protected_units(L_c: int, B: int, n_init: int, n_local: int) -> list[int]:
    """Units that overlap the first n_init or the last n_local tokens of a context.
    Section 3.2 keeps initial and local positions at full resolution (Section 4.1:
    1 initial block and 2 local blocks of 64 tokens in the paper's runs)."""
    nb = -(-L_c // B)
    prot = []
    for m in range(nb):
        a = m * B
        b = min(a + B, L_c)
        if a < n_init or b > L_c - n_local:
            prot.append(m)
    return prot


def budget_units(L_c: int, B: int, n_init: int, n_local: int, budget_bp: int) -> int:
    """Units kept in a context under a sequence budget given in basis points
    (1500 = 15 %): floor(budget * nb), never below the protected count, never above nb.
    (The paper's own count is dynamic, Eq. 2-3; the fixed budget mirrors its reported
    ~15 % sequence ratio, Table 1.)"""
    nb = -(-L_c // B)
    n_prot = len(protected_units(L_c, B, n_init, n_local))
    k = (budget_bp * nb) // 10000
    return max(n_prot, min(nb, k))


def select_units(u: np.ndarray, ctx_offsets, B: int, n_init: int, n_local: int, k_units) -> np.ndarray:
    """Per KV head and per context keep the protected units plus the best middle units.

    u: [Hkv, U_tot] unit scores; k_units[c] = units kept in context c, protected ones
    included.  Middle units are ranked by (score descending, index ascending) with a
    stable sort, so of equal scores the lower index wins.  Returns global unit ids,
    ascending, [Hkv, sum(k_units)]; context c's segment starts at sum(k_units[:c]).
    """
    u = np.asarray(u, dtype=F64)
    Hkv = u.shape[0]
    nb, unit_off = unit_layout(ctx_offsets, B)
    D = len(nb)
    S_u = int(sum(int(k) for k in k_units))
    sel = np.zeros((Hkv, S_u), dtype=np.int32)
    for h in range(Hkv):
        pos = 0
        for c in range(D):
            L_c = int(ctx_offsets[c + 1]) - int(ctx_offsets[c])
            prot = protected_units(L_c, B, n_init, n_local)
            k = int(k_units[c])
            assert len(prot) <= k <= nb[c], "k_units must lie in [n_prot, nb]"
            prot_set = set(prot)
            middle = [m for m in range(nb[c]) if m not in prot_set]
            # stable sort: score descending, then index ascending
            order = sorted(middle, key=lambda m: (-u[h, unit_off[c] + m], m))
            picked = order[: k - len(prot)]
            kept = sorted(prot + picked)
            for m in kept:
                sel[h, pos] = unit_off[c] + m
                pos += 1
    return sel


def kth_middle_score(u_row: np.ndarray, ctx_offsets, B: int, n_init: int, n_local: int, k_units, c: int):
    """Score of the last middle unit the oracle keeps in context c (None if it keeps no
    middle unit).  Used by the parity check's near-tie band, never by the method."""
    nb, unit_off = unit_layout(ctx_offsets, B)
    L_c = int(ctx_offsets[c + 1]) - int(ctx_offsets[c])
    prot = set(protected_units(L_c, B, n_init, n_local))
    middle = [m for m in range(nb[c]) if m not in prot]
    n_pick = int(k_units[c]) - len(prot)
    if n_pick <= 0 or not middle:
        return None
    vals = sorted((float(u_row[unit_off[c] + m]) for m in middle), reverse=True)
    return vals[n_pick - 1]


def units_to_tokens(sel_row: np.ndarray, ctx_offsets, B: int) -> np.ndarray:
    """Global unit ids -> global token ids, in the same order (context, then token,
    ascending when the unit ids ascend)."""
    nb, unit_off = unit_layout(ctx_offsets, B)
    toks = []
    for uid in sel_row:
        uid = int(uid)
        c = 0
        while not (unit_off[c] <= uid < unit_off[c + 1]):
            c += 1
        m = uid - unit_off[c]
        lo, hi = int(ctx_offsets[c]), int(ctx_offsets[c + 1])
        a = lo + m * B
        b = min(a + B, hi)
        toks.extend(range(a, b))
    return np.asarray(toks, dtype=np.int64)


# --------------------------------------------------------------------------------------
# Section 3.2 (end): the sparse cache = initial + selected + local, original order
# --------------------------------------------------------------------------------------
def compact(K: np.ndarray, V: np.ndarray, sel: np.ndarray, ctx_offsets, B: int, capacity: int | None = None):
    """Kc[h, slot, :] = K[h, tok(slot), :] (same for V); slots follow (context, token)
    ascending.  Returns (Kc, Vc, cache_len, inv_map) with inv_map[h, token] = slot or -1
    (the paper's "blank" position for a token this head did not keep).
    K, V: [Hkv, L_tot, d]; sel: [Hkv, S_u]."""
    K = np.asarray(K)
    V = np.asarray(V)
    Hkv, L_tot, d = K.shape
    toks0 = units_to_tokens(sel[0], ctx_offsets, B)
    S = len(toks0)
    cap = S if capacity is None else capacity
    assert cap >= S
    Kc = np.zeros((Hkv, cap, d), dtype=K.dtype)
    Vc = np.zeros((Hkv, cap, d), dtype=V.dtype)
    inv = np.full((Hkv, L_tot), -1, dtype=np.int32)
    for h in range(Hkv):
        toks = units_to_tokens(sel[h], ctx_offsets, B)
        assert len(toks) == S, "every head keeps the same number of tokens"
        for slot, t in enumerate(toks):
            Kc[h, slot] = K[h, t]
            Vc[h, slot] = V[h, t]
            inv[h, t] = slot
    return Kc, Vc, S, inv


# --------------------------------------------------------------------------------------
# Section 3.3: write recomputed rows back — Overwrite, or Fusion (Eq. 4)
# --------------------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (ties to even), returned as float64."""
    f32 = np.asarray(x, dtype=np.float32)
    bits = f32.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    rounded = ((bits + 0x7FFF + lsb) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).astype(F64)


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.asarray(x, dtype=np.float32).astype(F64)
    if dtype == "f64":
        return np.asarray(x, dtype=F64)
    raise ValueError(dtype)


def fuse_row(new: np.ndarray, old: np.ndarray) -> np.ndarray:
    """Eq. 4 for one row: theta = cos(new, old); result = theta*new + (1-theta)*old.
    theta = 1 when a norm is zero (the row is then simply replaced)."""
    c = _cos(new, old)
    theta = 1.0 if c is None else c
    return theta * new + (1.0 - theta) * old


def update(Kc: np.ndarray, Vc: np.ndarray, inv_map: np.ndarray, tok_ids, Knew: np.ndarray, Vnew: np.ndarray,
           mode: str, dtype: str = "f64"):
    """For every recomputed token r (global token id tok_ids[r], -1 = skip) and every KV
    head h that kept it (slot = inv_map[h, token] >= 0):
      overwrite: Kc[h, slot] = Knew[r, h];                     (Section 3.3 "Overwrite")
      fusion   : Kc[h, slot] = theta*Knew + (1-theta)*Kc_old   (Eq. 4), theta per row,
                 K and V each with their own theta; result rounded to the cache dtype.
    Kc, Vc: [Hkv, cap, d] float64 (modified copies are returned); Knew, Vnew: [R, Hkv, d]."""
    Kc = np.array(Kc, dtype=F64, copy=True)
    Vc = np.array(Vc, dtype=F64, copy=True)
    Knew = np.asarray(Knew, dtype=F64)
    Vnew = np.asarray(Vnew, dtype=F64)
    Hkv = Kc.shape[0]
    for r, tok in enumerate(tok_ids):
        tok = int(tok)
        if tok < 0:
            continue
        for h in range(Hkv):
            slot = int(inv_map[h, tok])
            if slot < 0:
                continue
            if mode == "overwrite":
                Kc[h, slot] = Knew[r, h]
                Vc[h, slot] = Vnew[r, h]
            elif mode == "fusion":
                Kc[h, slot] = round_to_dtype(fuse_row(Knew[r, h], Kc[h, slot]), dtype)
                Vc[h, slot] = round_to_dtype(fuse_row(Vnew[r, h], Vc[h, slot]), dtype)
            else:
                raise ValueError(mode)
    return Kc, Vc


# --------------------------------------------------------------------------------------
# Section 3.3 (end): incremental prefill / decode of the query over the new sparse cache
# --------------------------------------------------------------------------------------
def attention(Kc: np.ndarray, Vc: np.ndarray, cache_len: int, Q: np.ndarray,
              Kq: np.ndarray | None = None, Vq: np.ndarray | None = None, scale: float | None = None):
    """Grouped-query softmax attention of a query chunk over the compact cache.

    Kc, Vc: [Hkv, cap, d]; Q: [T_q, Hq, d]; optional Kq, Vq: [T_q, Hkv, d] are the chunk's
    own keys/values, appended at slots cache_len .. cache_len+T_q-1.
    Query token t sees every slot < cache_len and appended slots cache_len+t' with t' <= t.
    Returns (O [T_q, Hq, d], lse [Hq, T_q], Kc', Vc', new cache_len).
    """
    Kc = np.array(Kc, dtype=F64, copy=True)
    Vc = np.array(Vc, dtype=F64, copy=True)
    Q = np.asarray(Q, dtype=F64)
    T_q, Hq, d = Q.shape
    Hkv = Kc.shape[0]
    G = Hq // Hkv
    if scale is None or scale <= 0:
        scale = 1.0 / np.sqrt(d)
    n_app = 0
    if Kq is not None:
        n_app = T_q
        assert cache_len + T_q <= Kc.shape[1], "cache capacity too small for the appended chunk"
        for t in range(T_q):
            Kc[:, cache_len + t, :] = np.asarray(Kq, dtype=F64)[t]
            Vc[:, cache_len + t, :] = np.asarray(Vq, dtype=F64)[t]
    O = np.zeros((T_q, Hq, d), dtype=F64)
    lse = np.zeros((Hq, T_q), dtype=F64)
    for t in range(T_q):
        n_vis = cache_len + (t + 1 if n_app else 0)
        for hq in range(Hq):
            h = hq // G
            logits = scale * (Kc[h, :n_vis, :] @ Q[t, hq])
            m = logits.max()
            e = np.exp(logits - m)
            Z = e.sum()
            p = e / Z
            O[t, hq] = p @ Vc[h, :n_vis, :]
            lse[hq, t] = m + np.log(Z)
    return O, lse, Kc, Vc, cache_len + n_app


# --------------------------------------------------------------------------------------
# The whole path for one (layer, batch element), in the paper's order
# --------------------------------------------------------------------------------------
def sparsify(K, V, Q, Qloc, ctx_offsets, B, n_init, n_local, k_units, use_bias=True, capacity=None):
    """pool -> Eq. 1 -> GQA fold -> token scores -> unit scores -> select -> compact.
    Returns a dict with every intermediate so that tests can compare stage by stage."""
    Hkv = K.shape[0]
    Q_que = pool_query(Q)
    q_loc = pool_local(Qloc) if Qloc is not None else None
    D = len(ctx_offsets) - 1
    Qhat = personalized_query(Q_que, q_loc, use_bias)
    if Qhat.shape[0] == 1 and D > 1:
        Qhat = np.repeat(Qhat, D, axis=0)
    q = fold_gqa(Qhat, Hkv)
    s = token_scores(q, K, ctx_offsets)
    u = unit_scores(s, ctx_offsets, B)
    sel = select_units(u, ctx_offsets, B, n_init, n_local, k_units)
    Kc, Vc, S, inv = compact(K, V, sel, ctx_offsets, B, capacity)
    return dict(Q_que=Q_que, q_loc=q_loc, Qhat=Qhat, q=q, s=s, u=u, sel=sel, Kc=Kc, Vc=Vc, cache_len=S, inv_map=inv)


# --------------------------------------------------------------------------------------
# Section 3.2, Eq. 2 and Eq. 3: dynamic Top-P from anchor / max / min scores, then the
# cross-context Top-K.  (Widening beyond the fixed-budget selection above.)
# --------------------------------------------------------------------------------------
def anchor_score(u_row: np.ndarray, c: int, ctx_offsets, B: int, n_init: int, n_local: int) -> float:
    """s_anc of context c: the anchor vector is read as the mean key over the protected
    (initial + local) tokens, so its score is the token-count-weighted mean of the protected
    units' scores (unit scores are means over their tokens)."""
    nb, unit_off = unit_layout(ctx_offsets, B)
    L_c = int(ctx_offsets[c + 1]) - int(ctx_offsets[c])
    tot, cnt = 0.0, 0
    for m in protected_units(L_c, B, n_init, n_local):
        n_tok = min((m + 1) * B, L_c) - m * B
        tot += float(u_row[unit_off[c] + m]) * n_tok
        cnt += n_tok
    return tot / cnt if cnt else 0.0


def top_p_ratio(s_anc: float, s_max: float, s_min: float) -> float:
    """Eq. 2: P = (s_max - s_anc) / (s_max - s_min) if s_anc in (s_min, s_max], else 0."""
    if s_min < s_anc <= s_max:
        return (s_max - s_anc) / (s_max - s_min)
    return 0.0


def middle_units(L_c: int, B: int, n_init: int, n_local: int) -> list[int]:
    prot = set(protected_units(L_c, B, n_init, n_local))
    return [m for m in range(-(-L_c // B)) if m not in prot]


def top_p_per_head(u: np.ndarray, ctx_offsets, B: int, n_init: int, n_local: int,
                   max_units=None, min_units=None) -> np.ndarray:
    """P^(n)_doc-i for one layer (and batch element): [Hkv, D].  s_max / s_min are the scores of the
    caller's max / min blocks (global unit ids [D], from the offline analysis of Appendix A.1) or,
    when none are given, the largest / smallest middle-unit score.  A context without middle
    units gets 0."""
    u = np.asarray(u, dtype=F64)
    nb, unit_off = unit_layout(ctx_offsets, B)
    D = len(nb)
    P = np.zeros((u.shape[0], D), dtype=F64)
    for h in range(u.shape[0]):
        for c in range(D):
            L_c = int(ctx_offsets[c + 1]) - int(ctx_offsets[c])
            mid = middle_units(L_c, B, n_init, n_local)
            if not mid:
                continue
            vals = [float(u[h, unit_off[c] + m]) for m in mid]
            s_max = float(u[h, int(max_units[c])]) if max_units is not None else max(vals)
            s_min = float(u[h, int(min_units[c])]) if min_units is not None else min(vals)
            P[h, c] = top_p_ratio(anchor_score(u[h], c, ctx_offsets, B, n_init, n_local), s_max, s_min)
    return P


def consolidate_top_p(P_layers: np.ndarray) -> np.ndarray:
    """Eq. 3: P_doc-i = mean over the stable layers N* of P^(n)_doc-i.  P_layers: [|N*|, Hkv, D];
    the paper has no head index, so the KV heads are averaged too: one ratio per document."""
    P_layers = np.asarray(P_layers, dtype=F64)
    D = P_layers.shape[-1]
    out = np.zeros(D, dtype=F64)
    for c in range(D):
        tot = 0.0
        for n in range(P_layers.shape[0]):
            for h in range(P_layers.shape[1]):
                tot += P_layers[n, h, c]
        out[c] = tot / (P_layers.shape[0] * P_layers.shape[1])
    return out


def candidate_counts(P_doc: np.ndarray, ctx_offsets, B: int, n_init: int, n_local: int) -> list[int]:
    """Top-P of a document: floor(P * number of middle units) middle units."""
    out = []
    for c, P in enumerate(P_doc):
        L_c = int(ctx_offsets[c + 1]) - int(ctx_offsets[c])
        n_mid = len(middle_units(L_c, B, n_init, n_local))
        out.append(max(0, min(n_mid, int(np.floor(float(P) * n_mid + 1e-12)))))
    return out


def cross_context_select(u: np.ndarray, ctx_offsets, B: int, n_init: int, n_local: int, cand_counts):
    """Section 3.2, last paragraph.  Per KV head: in every context the cand_counts[c] best middle
    units are retrieved; their scores are min-max normalised inside their context
    ((u - min) / (max - min) over that context's middle units; 0 if max == min); the retrieved
    units of all contexts are compared and the best K = floor(total retrieved / D) are kept
    (equal normalised scores: lower global unit id first).  Protected units are always kept.
    Returns (sel [Hkv, S_u] ascending global unit ids, counts [Hkv, D] units kept per context)."""
    u = np.asarray(u, dtype=F64)
    Hkv = u.shape[0]
    nb, unit_off = unit_layout(ctx_offsets, B)
    D = len(nb)
    C = int(sum(int(c) for c in cand_counts))
    K = C // D
    prot_all = []
    for c in range(D):
        L_c = int(ctx_offsets[c + 1]) - int(ctx_offsets[c])
        prot_all.append([unit_off[c] + m for m in protected_units(L_c, B, n_init, n_local)])
    S_u = sum(len(p) for p in prot_all) + K
    sel = np.zeros((Hkv, S_u), dtype=np.int32)
    counts = np.zeros((Hkv, D), dtype=np.int32)
    for h in range(Hkv):
        pool = []                                   # (normalised score, global unit id)
        for c in range(D):
            L_c = int(ctx_offsets[c + 1]) - int(ctx_offsets[c])
            mid = middle_units(L_c, B, n_init, n_local)
            if not mid or cand_counts[c] == 0:
                continue
            vals = {m: float(u[h, unit_off[c] + m]) for m in mid}
            lo, hi = min(vals.values()), max(vals.values())
            order = sorted(mid, key=lambda m: (-vals[m], m))[: int(cand_counts[c])]
            for m in order:
                v = (vals[m] - lo) / (hi - lo) if hi > lo else 0.0
                pool.append((v, unit_off[c] + m))
        chosen = sorted(pool, key=lambda t: (-t[0], t[1]))[:K]
        kept = sorted([uid for _, uid in chosen] + [uid for p in prot_all for uid in p])
        sel[h] = kept
        for uid in kept:
            c = 0
            while not (unit_off[c] <= uid < unit_off[c + 1]):
                c += 1
            counts[h, c] += 1
    return sel, counts


# --------------------------------------------------------------------------------------
# Section 3.3 "Recomputation": blank-block alignment across layers and the two rules
# --------------------------------------------------------------------------------------
FLAG_KEPT = 1        # some KV head of this layer keeps the token (not a blank position)
FLAG_RECOMPUTE = 2   # the token's K/V of this layer are recomputed (rule 2, "when necessary")
FLAG_OUTPUT = 4      # this layer must also produce the token's output (rule 1: a higher layer recomputes it)
FLAG_PAD_REUSE = 8   # blank here, yet on the forward path: its prefilled K/V entry is used for the output


def align_layers(inv_map: np.ndarray, tok_ids: np.ndarray):
    """Pad -> merge -> recompute plan -> (the caller removes the padding again).

    inv_map [L, Hkv, L_tot]: slot of token t in the compact cache of (layer, head), -1 = blank.
    tok_ids [L, R]: tokens whose K/V should be recomputed at each layer (-1 = unused entry).

    A token is a blank position of layer n when no head of that layer keeps it.  Laying every
    layer over the union of all layers' kept tokens (the merged axis) aligns them; the blanks
    are the padding.  For layer n and token t:
      recompute  t is listed for layer n and layer n keeps it (a listed token that is blank at
                 layer n has no cache entry to refresh);
      output     some layer m > n recomputes t: computing t's K/V at layer m needs t's hidden
                 state, hence the outputs of every layer below m (rule 1);
      pad_reuse  output is needed, t is not recomputed here and is blank here: the forward pass
                 takes t's prefilled K/V entry (rule 2 reuses what exists).
    Returns (flags [L, L_tot] uint8, merged token ids ascending, per-layer ascending lists of
    the tokens that enter the layer's forward pass = recompute or output)."""
    inv_map = np.asarray(inv_map)
    tok_ids = np.asarray(tok_ids)
    L, Hkv, L_tot = inv_map.shape
    flags = np.zeros((L, L_tot), dtype=np.uint8)
    merged = []
    for t in range(L_tot):
        on_axis = False
        for n in range(L):
            kept = any(inv_map[n, h, t] >= 0 for h in range(Hkv))
            on_axis = on_axis or kept
            listed = any(int(x) == t for x in tok_ids[n])
            rec = listed and kept
            f = 0
            if kept:
                f |= FLAG_KEPT
            if rec:
                f |= FLAG_RECOMPUTE
            flags[n, t] = f
        if on_axis:
            merged.append(t)
    for t in range(L_tot):
        for n in range(L):
            higher = any(flags[m, t] & FLAG_RECOMPUTE for m in range(n + 1, L))
            if higher:
                flags[n, t] |= FLAG_OUTPUT
                if not (flags[n, t] & FLAG_RECOMPUTE) and not (flags[n, t] & FLAG_KEPT):
                    flags[n, t] |= FLAG_PAD_REUSE
    run = []
    for n in range(L):
        run.append(np.asarray([t for t in range(L_tot) if flags[n, t] & (FLAG_RECOMPUTE | FLAG_OUTPUT)],
                              dtype=np.int64))
    return flags, np.asarray(merged, dtype=np.int64), run


# --------------------------------------------------------------------------------------
# Section 3.2: "each block is represented by the mean vector of its constituent token caches"
# --------------------------------------------------------------------------------------
def block_means(K: np.ndarray, ctx_offsets, B: int, dtype: str | None = None) -> np.ndarray:
    """Kbar[h, u, :] = mean of K[h, t, :] over the tokens t of unit u (a short tail unit averages
    the tokens it has).  K: [Hkv, L_tot, d] float64 -> [Hkv, U_tot, d]; `dtype` ("bf16" / "f32")
    rounds the result once to the storage type of the representative cache, None keeps float64.
    Scoring a query against Kbar with `token_scores` over the unit offsets gives the block scores."""
    K = np.asarray(K, dtype=F64)
    nb, unit_off = unit_layout(ctx_offsets, B)
    Hkv, _, d = K.shape
    out = np.zeros((Hkv, unit_off[-1], d), dtype=F64)
    for h in range(Hkv):
        for c in range(len(nb)):
            lo, hi = int(ctx_offsets[c]), int(ctx_offsets[c + 1])
            for m in range(nb[c]):
                a = lo + m * B
                b = min(a + B, hi)
                acc = np.zeros(d, dtype=F64)
                for t in range(a, b):
                    acc += K[h, t]
                out[h, unit_off[c] + m] = acc / (b - a)
    return out if dtype is None else round_to_dtype(out, dtype)

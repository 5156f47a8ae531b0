"""Shared test helpers: run the CUDA library on a workload, run the oracle on the same stored
values, and compare stage by stage with the acceptance rules stated in each function."""
from __future__ import annotations

import numpy as np
import torch

from oracle import samkv_oracle as O
from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import synth


CANARY, CANARY_WORDS = 12345, 64


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact up-conversion of stored bf16 / fp32 values."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_k_units(w) -> list:
    return [O.budget_units(n, w.block_size, w.n_init, w.n_local, w.budget_bp) for n in w.ctx_lens]


ATTN_SHARE_SM = False      # set by a fixture: every DeviceRun then asks for the SM-sharing attention kernel


class DeviceRun:
    """One pass of the library over a workload; keeps every intermediate tensor."""

    def __init__(self, w, inp, k_units=None, use_bias=True, extra_capacity=None, with_qloc=True):
        self.w, self.inp = w, inp
        self.shape = B.Shape.from_workload(w)
        self.k_units = list(k_units) if k_units is not None else B.samkv_budget_units(self.shape, w.budget_bp)
        prot, self.U_tot, self.S = B.samkv_layout(self.shape, self.k_units)
        self.n_prot = prot
        extra = w.q_tokens + w.decode_steps if extra_capacity is None else extra_capacity
        self.capacity = self.S + extra
        dev = inp["K"].device
        L, Bt, Hkv, d = w.n_layers, w.batch, w.n_kv_heads, w.head_dim
        self.handle = B.Handle(self.shape, max(w.q_tokens, 1), self.capacity)
        if ATTN_SHARE_SM:                      # tests of the attention kernel that leaves room on its SM
            B.samkv_attn_share_sm(self.handle, True)
        # outputs sit in front of canary words that no kernel may touch (checked by poll())
        self._guarded = []

        def guarded(shape, dtype, fill=None):
            n = 1
            for v in shape:
                n *= v
            flat = torch.empty(n + CANARY_WORDS, dtype=dtype, device=dev)
            flat[n:] = CANARY
            if fill is not None:
                flat[:n] = fill
            self._guarded.append(flat[n:])
            return flat[:n].view(shape)

        self.scores = guarded((L, Bt, Hkv, self.U_tot), torch.float32)
        self.qhat = guarded((L, Bt, w.n_ctx, Hkv, d), torch.float32)
        self.sel = guarded((L, Bt, Hkv, sum(self.k_units)), torch.int32, fill=-7)
        self.Kc = torch.zeros((L, Bt, Hkv, self.capacity, d), dtype=w.torch_dtype, device=dev)
        self.Vc = torch.zeros_like(self.Kc)
        self.cache_len = torch.zeros((L, Bt), dtype=torch.int32, device=dev)
        self.inv_map = torch.zeros((L, Bt, Hkv, w.l_tot), dtype=torch.int32, device=dev)
        self.use_bias = use_bias
        self.with_qloc = with_qloc

    def sparsify(self):
        w, inp = self.w, self.inp
        B.samkv_score(self.handle, self.shape, inp["K"], inp["Q"], w.q_tokens,
                      inp["Qloc"] if self.with_qloc else None, inp["Qloc"].shape[3], int(self.use_bias), self.scores,
                      self.qhat)
        B.samkv_select(self.handle, self.shape, self.scores, self.k_units, self.sel)
        B.samkv_compact(self.handle, self.shape, inp["K"], inp["V"], self.sel, self.k_units, self.Kc, self.Vc,
                        self.capacity, self.cache_len, self.inv_map)
        return self

    def update(self, tok_ids, Knew, Vnew, mode):
        B.samkv_update(self.handle, self.shape, self.Kc, self.Vc, self.capacity, self.inv_map, tok_ids,
                       tok_ids.shape[1], Knew, Vnew, mode)
        return self

    def attn(self, layer, Q, Kq=None, Vq=None, scale=0.0, want_lse=True):
        Bt, T_q, Hq, d = Q.shape
        Oo = torch.empty_like(Q)
        lse = torch.empty((Bt, Hq, T_q), dtype=torch.float32, device=Q.device) if want_lse else None
        B.samkv_attn(self.handle, self.shape, layer, self.Kc, self.Vc, self.capacity, self.cache_len, Q, T_q, Kq, Vq,
                     scale, Oo, lse)
        return Oo, lse

    def poll(self):
        status = B.samkv_poll_status(self.handle)        # synchronises the stream
        for tail in self._guarded:
            assert bool((tail == CANARY).all()), "a kernel wrote past the end of an output"
        return status


def oracle_scores(w, inp, l, b, use_bias=True, with_qloc=True):
    """Oracle stages up to unit scores for one (layer, batch element)."""
    Q = to_f64(inp["Q"][l, b])
    Qloc = to_f64(inp["Qloc"][l, b]) if with_qloc else None
    K = to_f64(inp["K"][l, b])
    Q_que = O.pool_query(Q)
    q_loc = O.pool_local(Qloc) if Qloc is not None else None
    Qhat = O.personalized_query(Q_que, q_loc, use_bias)
    if Qhat.shape[0] == 1 and w.n_ctx > 1:
        Qhat = np.repeat(Qhat, w.n_ctx, axis=0)
    q = O.fold_gqa(Qhat, w.n_kv_heads)
    s = O.token_scores(q, K, w.ctx_offsets)
    u = O.unit_scores(s, w.ctx_offsets, w.block_size)
    return q, s, u


def check_scores(w, run: DeviceRun, l, b, q, u, K64=None):
    """Scores and q^ are diagnostics: |gpu - oracle| <= 1e-5 * ||q|| * ||K row|| (bounded here by the
    largest row norm of the slab), q^ to 1e-5 relative to its norm."""
    qg = run.qhat[l, b].cpu().double().numpy()                           # [D, Hkv, d]
    for c in range(w.n_ctx):
        for h in range(w.n_kv_heads):
            nq = np.linalg.norm(q[c, h])
            assert np.abs(qg[c, h] - q[c, h]).max() <= 1e-5 * max(nq, 1e-30), f"qhat mismatch l{l} b{b} c{c} h{h}"
    ug = run.scores[l, b].cpu().double().numpy()
    if K64 is None:
        K64 = to_f64(run.inp["K"][l, b])
    knorm = np.sqrt((K64 ** 2).sum(-1)).max(axis=1)                       # [Hkv]
    nb, off = O.unit_layout(w.ctx_offsets, w.block_size)
    for c in range(w.n_ctx):
        for h in range(w.n_kv_heads):
            tol = 1e-5 * np.linalg.norm(q[c, h]) * knorm[h]
            err = np.abs(ug[h, off[c]:off[c + 1]] - u[h, off[c]:off[c + 1]]).max()
            assert err <= tol, f"score mismatch l{l} b{b} c{c} h{h}: {err} > {tol}"


def check_selection(w, k_units, sel_gpu_lb: np.ndarray, u: np.ndarray, where=""):
    """Index sets must match the oracle exactly, lower index winning ties, except at units whose
    oracle score lies within 1e-5 relative of the oracle's k-th middle score; counts, order and the
    protected units must always be right.  Returns the number of (head, context) sets that differed."""
    nb, off = O.unit_layout(w.ctx_offsets, w.block_size)
    sel_or = O.select_units(u, w.ctx_offsets, w.block_size, w.n_init, w.n_local, k_units)
    n_diff = 0
    for h in range(u.shape[0]):
        row = sel_gpu_lb[h]
        assert np.all(np.diff(row) > 0), f"{where} h{h}: ids not strictly ascending"
        pos = 0
        for c in range(w.n_ctx):
            k = int(k_units[c])
            g = row[pos:pos + k]
            o = sel_or[h, pos:pos + k]
            pos += k
            assert g.min() >= off[c] and g.max() < off[c + 1], f"{where} h{h} c{c}: id outside its context"
            prot = set(off[c] + m for m in O.protected_units(w.ctx_lens[c], w.block_size, w.n_init, w.n_local))
            assert prot <= set(g.tolist()), f"{where} h{h} c{c}: protected unit missing"
            if np.array_equal(g, o):
                continue
            n_diff += 1
            u_k = O.kth_middle_score(u[h], w.ctx_offsets, w.block_size, w.n_init, w.n_local, k_units, c)
            band = 1e-5 * abs(u_k)
            for uid in set(g.tolist()) ^ set(o.tolist()):
                assert abs(u[h, uid] - u_k) <= band, (f"{where} h{h} c{c}: unit {uid} differs outside the tie band "
                                                      f"(score {u[h, uid]}, k-th {u_k})")
    return n_diff


def check_compact(w, run: DeviceRun, l, b, sel_lb: np.ndarray):
    """Bit-exact gather with the GPU's own index set; inverse map round trip; cache_len."""
    K = run.inp["K"][l, b].cpu()
    V = run.inp["V"][l, b].cpu()
    Kc = run.Kc[l, b].cpu()
    Vc = run.Vc[l, b].cpu()
    inv = run.inv_map[l, b].cpu().numpy()
    assert int(run.cache_len[l, b]) == run.S
    for h in range(w.n_kv_heads):
        toks = O.units_to_tokens(sel_lb[h], w.ctx_offsets, w.block_size)
        assert len(toks) == run.S
        idx = torch.from_numpy(toks)
        assert torch.equal(Kc[h, :run.S].view(torch.uint8), K[h, idx].view(torch.uint8)), f"Kc l{l} b{b} h{h}"
        assert torch.equal(Vc[h, :run.S].view(torch.uint8), V[h, idx].view(torch.uint8)), f"Vc l{l} b{b} h{h}"
        exp = np.full(w.l_tot, -1, dtype=np.int32)
        exp[toks] = np.arange(run.S, dtype=np.int32)
        assert np.array_equal(inv[h], exp), f"inv_map l{l} b{b} h{h}"
    # slots beyond S untouched (the buffers were zero-filled)
    assert not Kc[:, run.S:].to(torch.float32).any() and not Vc[:, run.S:].to(torch.float32).any()


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bfloat16 at |x| (8 significant bits)."""
    ax = np.maximum(np.abs(x), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def check_update(w, Kc_before, Vc_before, Kc_after, Vc_after, inv_lb, tok_ids_l, Knew_lb, Vnew_lb, mode):
    """Overwrite: bit-exact.  Fusion: the GPU forms theta and the blend in fp32, the oracle in fp64, and
    both round the row to the cache dtype, so an element may differ by one unit in the last place of
    the oracle value, plus the fp32 error of the blend, which scales with the operands (not with a
    result that may have cancelled): 1e-5 * (|new| + |old|) per element.  fp32 caches: 1e-5 of the row
    norm.  Untouched slots must be bit-identical."""
    mode_name = "overwrite" if mode == B.SAMKV_UPDATE_OVERWRITE else "fusion"
    Kb, Vb = to_f64(Kc_before), to_f64(Vc_before)
    Kn, Vn = to_f64(Knew_lb), to_f64(Vnew_lb)
    Ko, Vo = O.update(Kb, Vb, inv_lb, tok_ids_l, Kn, Vn, mode_name, dtype=w.dtype)
    Kg, Vg = to_f64(Kc_after), to_f64(Vc_after)
    touched = np.zeros(Kg.shape[:2], dtype=bool)
    mag_k, mag_v = np.zeros_like(Kg), np.zeros_like(Vg)
    for r, tok in enumerate(tok_ids_l):
        if tok >= 0:
            for h in range(Kg.shape[0]):
                slot = inv_lb[h, tok]
                if slot >= 0:
                    touched[h, slot] = True
                    mag_k[h, slot] = np.abs(Kn[r, h]) + np.abs(Kb[h, slot])
                    mag_v[h, slot] = np.abs(Vn[r, h]) + np.abs(Vb[h, slot])
    assert np.array_equal(Kg[~touched], Kb[~touched]) and np.array_equal(Vg[~touched], Vb[~touched])
    if mode_name == "overwrite":
        assert np.array_equal(Kg, Ko) and np.array_equal(Vg, Vo)
        return
    for got, exp, mag in ((Kg, Ko, mag_k), (Vg, Vo, mag_v)):
        if w.dtype == "bf16":
            tol = bf16_ulp(exp) + 1e-5 * mag
            assert np.all(np.abs(got - exp)[touched] <= tol[touched])
        else:
            nrm = np.sqrt((exp ** 2).sum(-1, keepdims=True))
            assert np.all(np.abs(got - exp)[touched] <= 1e-5 * nrm[touched] + 1e-30)


def attn_tolerance(w) -> float:
    """max-abs error bound on attention outputs: 2e-2 for bf16 inputs (fp32 accumulation), 1e-4 for fp32."""
    return 2e-2 if w.dtype == "bf16" else 1e-4


# The absolute bf16 bound is loose where the outputs are small (with N(0,1) values and thousands of visible slots
# |O| is a few hundredths), so a second, relative bound goes with it: per query head, the largest error may be at
# most 2^-6 of the largest oracle output of that head.  The kernels round P and O to bf16 (2^-9 relative each) and
# accumulate in fp32, so errors of about 2^-8 of the head's largest output are expected; 2^-6 leaves a factor of
# four and still fails a result that is off by a few percent.  The softmax denominator is summed in fp32 over the
# bf16-rounded probabilities (the values the tensor core multiplies with V), so lse can be off by log(1 + 2^-9) =
# 2e-3 when one probability dominates; its bound is 2^-8.
ATTN_REL_BOUND_BF16 = 2.0 ** -6
LSE_BOUND_BF16 = 2.0 ** -8
OBSERVED = {"attn_rel": 0.0, "lse": 0.0}      # largest values seen in this process (printed by the tests that ask)


def check_attention(w, Kc_lb, Vc_lb, cache_len, Q_b, Kq_b, Vq_b, O_gpu_b, lse_gpu_b=None, scale=None, t_sample=None):
    """Oracle attention on the GPU's own compact cache values; optional sampling of query tokens
    (only when nothing is appended, so that visibility does not depend on the token index)."""
    Kc64, Vc64 = to_f64(Kc_lb), to_f64(Vc_lb)
    Q64 = to_f64(Q_b)
    if t_sample is not None:
        assert Kq_b is None
        Q64 = Q64[t_sample]
    out, lse, K2, V2, n = O.attention(Kc64, Vc64, cache_len, Q64, None if Kq_b is None else to_f64(Kq_b),
                                      None if Vq_b is None else to_f64(Vq_b), scale)
    got = to_f64(O_gpu_b)
    if t_sample is not None:
        got = got[t_sample]
    err = np.abs(got - out).max()
    assert err <= attn_tolerance(w), f"attention max-abs error {err}"
    if w.dtype == "bf16":
        # out, got: [T, Hq, d] -> per query head over tokens and elements
        head_err = np.abs(got - out).max(axis=(0, 2))
        head_max = np.abs(out).max(axis=(0, 2))
        rel = float((head_err / np.maximum(head_max, 1e-30)).max())
        OBSERVED["attn_rel"] = max(OBSERVED["attn_rel"], rel)
        assert rel <= ATTN_REL_BOUND_BF16, f"attention error {rel:.3e} of a head's largest output (bound 2^-6)"
    if lse_gpu_b is not None:
        lg = to_f64(lse_gpu_b)
        if t_sample is not None:
            lg = lg[:, t_sample]
        lse_err = float(np.abs(lg - lse).max())
        if w.dtype == "bf16":
            OBSERVED["lse"] = max(OBSERVED["lse"], lse_err)
        assert lse_err <= (LSE_BOUND_BF16 if w.dtype == "bf16" else 1e-4), f"lse error {lse_err}"
    return err, K2, V2, n

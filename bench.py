#!/usr/bin/env python
"""Benchmark of the SamKV hot path on B200.

One step = one pass of the whole path (score -> select -> compact -> update(fusion) -> attention for
every layer) over one synthetic request batch of the `cfg2` workload (Llama-3-8B attention shape,
32 layers, 20 contexts x 1536 tokens, batch 4, 64 query tokens, 15 % budget, 15 % of the kept
tokens recomputed).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl samkv|reference]

Under torchrun every rank processes its own batch (weak scaling, no data-path collective); the
reported time is the maximum over ranks of the CUDA-event time of the K timed steps.
`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2508_11661_b200 import synth

METRIC = "context_kv_tokens_scored_and_attended_per_s"
UNIT = "tokens/s"
HBM_NOMINAL_GBS = 8000.0
HBM_FALLBACK_GBS = 6650.0

# kernels each C-ABI call enqueues (memsets are not counted)
KERNELS_PER_CALL = {"score": 2, "select": 1, "compact": 1, "update": 1}      # samkv_attn: asked from the library


def score_kernel_dram_bytes_per_row():
    """DRAM bytes per scored key row of score_stream_kernel (dram read + write of one launch / rows of that launch),
    from the ncu capture summarised under profiles/; traffic grows in proportion to the rows (no reuse), so a full
    launch is rows x this figure.  Kept in a small file beside the profile it came from."""
    p = os.path.join(ROOT, "profiles", "score_stream_kernel_dram_bytes.json")
    try:
        with open(p) as f:
            return float(json.load(f)["dram_bytes_per_row"])
    except Exception:
        return None


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": HBM_FALLBACK_GBS}, "fallback"


# --------------------------------------------------------------------------------------------------
# algorithmic bytes of one step (what the method itself must move)
# --------------------------------------------------------------------------------------------------
def algorithmic_bytes(w, S: int, R: int, fusion: bool = True, kept_rows=None) -> dict:
    """kept_rows: (layer, batch, recomputed token, KV head) combinations whose head kept the token.  Every listed
    combination reads its new K and V row; only the kept ones read the old rows (fusion) and write the result.
    None charges every combination as kept.  The inverse map (4 B per token, memset + scatter) and the scores /
    index lists are not charged."""
    e = w.elem_bytes
    row = w.head_dim * e
    slabs = w.n_layers * w.batch * w.n_kv_heads
    kbytes = slabs * w.l_tot * row
    score = kbytes                                        # every K row once
    gather = slabs * S * row * 4                          # read K,V rows, write Kc,Vc rows
    listed = w.n_layers * w.batch * R * w.n_kv_heads
    kept = listed if kept_rows is None else int(kept_rows)
    upd = (2 * listed + (4 if fusion else 2) * kept) * row
    attn = slabs * (S + w.q_tokens) * row * 2             # attention reads Kc,Vc (cache + chunk)
    # decode step i reads the cache as it stands then: S + T_q + i slots (+ its own row)
    dec = sum(slabs * (S + w.q_tokens + i + 1) * row * 2 for i in range(w.decode_steps))
    return {"score": score, "compact": gather, "update": upd, "attn": attn, "decode": dec,
            "total": score + gather + upd + attn + dec}


# --------------------------------------------------------------------------------------------------
# clock sampling during the timed region
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.gpu_index)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def window_open(self):
        import datetime
        self.t0 = datetime.datetime.now()

    def window_close(self):
        import datetime
        self.t1 = datetime.datetime.now()

    def stop(self) -> dict:
        """Median SM clock and throttle reasons over the samples taken inside [window_open, window_close]
        (all samples if the window caught none: the sampler's period is 50 ms)."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 9:
                        continue
                    try:
                        ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                        rows.append((ts, float(parts[1]), float(parts[2]), parts[5:9]))
                    except ValueError:
                        continue
            os.unlink(self.path)
        except Exception:
            pass
        t0, t1 = getattr(self, "t0", None), getattr(self, "t1", None)
        inside = [r for r in rows if t0 is not None and t1 is not None and t0 <= r[0] <= t1 + datetime.timedelta(milliseconds=60)]
        use = inside if inside else rows
        reasons = set()
        for r in use:
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if use:
            out.update(sm_mhz=float(np.median([r[1] for r in use])), sm_max_mhz=float(max(r[2] for r in use)),
                       reasons=sorted(reasons), samples=len(use), samples_in_timed_region=len(inside))
        return out


# --------------------------------------------------------------------------------------------------
# the GPU arm
# --------------------------------------------------------------------------------------------------
ATTN_SHARE_SM = "auto"      # --attn-share-sm auto|on|off: which prefill attention kernel the overlapped schedule uses


class Pipeline:
    """Device-resident state of one request batch and the calls of one step."""

    def __init__(self, w, device, seed_offset=0):
        from paper_2508_11661_b200 import binding as B
        self.B = B
        self.w = w = w.replace(seed=w.seed + seed_offset)
        self.dev = device
        self.inp = synth.make_inputs(w, device)
        self.shape = B.Shape.from_workload(w)
        self.k_units = B.samkv_budget_units(self.shape, w.budget_bp)
        _, self.U_tot, self.S = B.samkv_layout(self.shape, self.k_units)
        self.capacity = self.S + w.q_tokens + w.decode_steps
        L, Bt, Hkv, d = w.n_layers, w.batch, w.n_kv_heads, w.head_dim
        self.handle = B.Handle(self.shape, w.q_tokens, self.capacity)
        # attention runs on its own high-priority stream with its own handle (own split-partial scratch), so
        # that the tensor-bound attention of one layer group overlaps the HBM-bound gather of the next
        self.shape1 = B.Shape.from_workload(w, n_layers=1)
        # Its kernels run next to the gather and update of the following layers.  samkv_attn_share_sm asks for the
        # attention kernel that leaves registers and shared memory on every SM (slower alone); whether that pays
        # depends on the shape, so choose_attention_kernel() times both during warm-up unless the flag fixes it.
        self.attn_share_sm = (ATTN_SHARE_SM == "on")
        self.schedule_trials = {}
        self.fused_select = False
        self.attn_stream = torch.cuda.Stream(device=device, priority=-1)
        # one attention call per group of layers (samkv_attn_layers); a handle per group count, because its workspace
        # is sized for the group's requests
        self._attn_handles = {}
        self.set_groups(8 if (w.n_layers % 8 == 0 and w.decode_steps == 0) else 1)
        self.scores = torch.empty((L, Bt, Hkv, self.U_tot), dtype=torch.float32, device=device)
        self.sel = torch.empty((L, Bt, Hkv, sum(self.k_units)), dtype=torch.int32, device=device)
        self.Kc = torch.zeros((L, Bt, Hkv, self.capacity, d), dtype=w.torch_dtype, device=device)
        self.Vc = torch.zeros_like(self.Kc)
        self.cache_len = torch.zeros((L, Bt), dtype=torch.int32, device=device)
        self.inv_map = torch.empty((L, Bt, Hkv, w.l_tot), dtype=torch.int32, device=device)
        self.O = torch.empty((L, Bt, w.q_tokens, w.n_q_heads, d), dtype=w.torch_dtype, device=device)
        self.R = 0
        self.update_kept_rows = None
        self.tok_ids = self.Knew = self.Vnew = None
        self.t_loc = self.inp["Qloc"].shape[3]
        self.decode_graph = None
        if w.decode_steps > 0:      # one query token per step and batch element, appended to the compact cache
            g = torch.Generator(device=device).manual_seed(w.seed + 99)
            n = w.decode_steps
            self.dq = torch.randn((n, Bt, 1, w.n_q_heads, d), generator=g, device=device).to(w.torch_dtype)
            self.dk = torch.randn((n, Bt, 1, Hkv, d), generator=g, device=device).to(w.torch_dtype)
            self.dv = torch.randn((n, Bt, 1, Hkv, d), generator=g, device=device).to(w.torch_dtype)
            self.dO = torch.empty_like(self.dq)

    def prepare_recompute(self):
        """Recompute list: R = 15 % of the kept tokens, drawn from what KV head 0 kept (needs one selection pass)."""
        w, B = self.w, self.B
        if w.recompute_share_bp <= 0:
            return
        self.sparsify()
        torch.cuda.synchronize()
        inv0 = self.inv_map[:, :1, 0, :]                               # [L, 1, L_tot] slots of head 0, batch 0
        toks0 = torch.stack([torch.nonzero(inv0[l, 0] >= 0).flatten() for l in range(w.n_layers)])[:, None, :]
        self.R = (w.recompute_share_bp * self.S) // 10000
        self.tok_ids, self.Knew, self.Vnew = synth.make_recompute(w, self.inp["K"], self.inp["V"], toks0, self.R)
        # rows the update really touches: heads other than head 0 keep only part of the listed tokens
        kept = 0
        for l in range(w.n_layers):
            kept += int((self.inv_map[l][:, :, self.tok_ids[l].long()] >= 0).sum())
        self.update_kept_rows = kept

    def attn_handle_for(self, groups: int):
        B, w = self.B, self.w
        if groups not in self._attn_handles:
            wide = B.Shape.from_workload(w.replace(batch=w.batch * (w.n_layers // groups)), n_layers=1)
            self._attn_handles[groups] = B.Handle(wide, w.q_tokens, self.capacity)
        return self._attn_handles[groups]

    def set_groups(self, groups: int):
        """The schedule's layer groups: 1 = everything in order on one stream with one attention call for all layers;
        g > 1 = gather + update of a group beside the attention of the previous groups."""
        self.groups = groups
        self.per_group = self.w.n_layers // groups
        self.handle_attn = self.attn_handle_for(groups)
        self.B.samkv_attn_share_sm(self.handle_attn, self.attn_share_sm if groups > 1 else False)

    def choose_schedule(self, steps: int = 3):
        """Warm-up time only: the step with 1, 2, 4 or 8 layer groups and, where groups overlap, with either prefill
        attention kernel; the fastest combination stays.  --attn-share-sm on|off fixes the kernel."""
        w = self.w
        if w.n_layers % 8 != 0 or w.decode_steps > 0:
            return
        shares = {"auto": (False, True), "on": (True,), "off": (False,)}[ATTN_SHARE_SM]
        best = None
        for groups, fused in ((1, False), (1, True), (2, False), (4, False), (8, False)):
            for share in (shares if groups > 1 else (False,)):
                self.attn_share_sm = share
                self.fused_select = fused
                self.set_groups(groups)
                for _ in range(2):
                    self.step()
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(steps):
                    self.step()
                b.record()
                torch.cuda.synchronize()
                ms = a.elapsed_time(b) / steps
                self.schedule_trials[f"{groups} groups" + (", sharing kernel" if share else "") +
                                     (", fused select+compact" if fused else "")] = ms
                if best is None or ms < best[0]:
                    best = (ms, groups, share, fused)
        self.attn_share_sm = best[2]
        self.fused_select = best[3]
        self.set_groups(best[1])

    def attn_group(self, g: int):
        """Attention of layer group g in one call (every layer's query chunk is available up front, as for the other
        phases, which take all layers per call)."""
        B, inp, w = self.B, self.inp, self.w
        n = self.per_group
        sl = slice(g * n, (g + 1) * n)
        B.samkv_attn_layers(self.handle_attn, self.shape, g * n, n, self.Kc, self.Vc, self.capacity, self.cache_len,
                            inp["Qa"][sl], w.q_tokens, inp["Kq"][sl], inp["Vq"][sl], 0.0, self.O[sl])

    def attn_all(self):
        """Attention of all layers in one call with the default kernel (the in-order phase table)."""
        B, inp, w = self.B, self.inp, self.w
        h = self.attn_handle_for(1)
        B.samkv_attn_share_sm(h, False)
        B.samkv_attn_layers(h, self.shape, 0, w.n_layers, self.Kc, self.Vc, self.capacity, self.cache_len, inp["Qa"],
                            w.q_tokens, inp["Kq"], inp["Vq"], 0.0, self.O)

    def sparsify(self):
        B, inp, w = self.B, self.inp, self.w
        B.samkv_score(self.handle, self.shape, inp["K"], inp["Q"], w.q_tokens, inp["Qloc"], self.t_loc, 1, self.scores)
        B.samkv_select(self.handle, self.shape, self.scores, self.k_units, self.sel)
        B.samkv_compact(self.handle, self.shape, inp["K"], inp["V"], self.sel, self.k_units, self.Kc, self.Vc,
                        self.capacity, self.cache_len, self.inv_map)

    def step(self, ev=None, overlap=True, attention_all_layers=False, fused_select=None):
        """One pass of the whole path.  `ev` (optional) collects CUDA events at phase boundaries.

        overlap=True (the timed schedule): scoring and selection of all layers first; then, per group of layers,
        compaction + update on the current stream while attention of the previous groups runs on a second,
        higher-priority stream (the gather kernels use no shared memory, so their CTAs share SMs with the
        attention CTAs).  overlap=False runs everything in order on one stream (per-phase timing)."""
        B, inp, w = self.B, self.inp, self.w
        main = torch.cuda.current_stream()

        def mark(name):
            if ev is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record()
                ev.append((name, e))

        mark("start")
        if overlap == "scan" and self.groups > 1:
            # Alternative schedule, measured beside the timed one: every phase group by group, so that the HBM-bound
            # scan (scoring, selection, gather, update) of group g + 1 runs while the tensor-bound attention of
            # group g is on the second stream.
            per = w.n_layers // self.groups
            shape_g = B.Shape.from_workload(w, n_layers=per)
            side = self.attn_stream
            side.wait_stream(main)
            for g in range(self.groups):
                sl = slice(g * per, (g + 1) * per)
                B.samkv_score(self.handle, shape_g, inp["K"][sl], inp["Q"][sl], w.q_tokens, inp["Qloc"][sl], self.t_loc, 1,
                              self.scores[sl])
                B.samkv_select(self.handle, shape_g, self.scores[sl], self.k_units, self.sel[sl])
                B.samkv_compact(self.handle, shape_g, inp["K"][sl], inp["V"][sl], self.sel[sl], self.k_units, self.Kc[sl],
                                self.Vc[sl], self.capacity, self.cache_len[sl], self.inv_map[sl])
                if self.R > 0:
                    B.samkv_update(self.handle, shape_g, self.Kc[sl], self.Vc[sl], self.capacity, self.inv_map[sl],
                                   self.tok_ids[sl], self.R, self.Knew[sl], self.Vnew[sl], B.SAMKV_UPDATE_FUSION)
                ready = torch.cuda.Event()
                ready.record(main)
                with torch.cuda.stream(side):
                    side.wait_event(ready)
                    self.attn_group(g)
            main.wait_stream(side)
            mark("scan_overlapped_with_attn")
            return
        B.samkv_score(self.handle, self.shape, inp["K"], inp["Q"], w.q_tokens, inp["Qloc"], self.t_loc, 1, self.scores)
        mark("score")
        fused = (self.fused_select if fused_select is None else fused_select) and not (overlap and self.groups > 1)
        if not fused:
            B.samkv_select(self.handle, self.shape, self.scores, self.k_units, self.sel)
            mark("select")
        if overlap and self.groups > 1:
            per = w.n_layers // self.groups
            shape_g = B.Shape.from_workload(w, n_layers=per)
            side = self.attn_stream
            side.wait_stream(main)
            for g in range(self.groups):
                sl = slice(g * per, (g + 1) * per)
                # (the fused samkv_select_compact is 0.07 ms faster than select + compact on its own, but its larger
                # CTAs lose more next to the attention kernels than that: 3.49 against 3.38 ms per step)
                B.samkv_compact(self.handle, shape_g, inp["K"][sl], inp["V"][sl], self.sel[sl], self.k_units, self.Kc[sl],
                                self.Vc[sl], self.capacity, self.cache_len[sl], self.inv_map[sl])
                if self.R > 0:
                    B.samkv_update(self.handle, shape_g, self.Kc[sl], self.Vc[sl], self.capacity, self.inv_map[sl],
                                   self.tok_ids[sl], self.R, self.Knew[sl], self.Vnew[sl], B.SAMKV_UPDATE_FUSION)
                ready = torch.cuda.Event()
                ready.record(main)
                with torch.cuda.stream(side):
                    side.wait_event(ready)
                    self.attn_group(g)
            main.wait_stream(side)
            mark("gather_update_attn_overlapped")
            return
        if fused:       # selection and gather of a (slab, context) by one CTA: no second launch, unit list not re-read
            B.samkv_select_compact(self.handle, self.shape, self.scores, self.k_units, inp["K"], inp["V"], self.sel,
                                   self.Kc, self.Vc, self.capacity, self.cache_len, self.inv_map)
            mark("select_compact")
        else:
            B.samkv_compact(self.handle, self.shape, inp["K"], inp["V"], self.sel, self.k_units, self.Kc, self.Vc,
                            self.capacity, self.cache_len, self.inv_map)
            mark("compact")
        if self.R > 0:
            B.samkv_update(self.handle, self.shape, self.Kc, self.Vc, self.capacity, self.inv_map, self.tok_ids, self.R,
                           self.Knew, self.Vnew, B.SAMKV_UPDATE_FUSION)
        mark("update")
        if attention_all_layers and self.groups > 1:
            self.attn_all()
        else:
            for g in range(self.groups):
                self.attn_group(g)
        mark("attn")
        if w.decode_steps > 0:
            self.decode()
            mark("decode")

    def decode_eager(self):
        B, w = self.B, self.w
        for l in range(w.n_layers):
            for i in range(w.decode_steps):
                B.samkv_attn(self.handle, self.shape, l, self.Kc, self.Vc, self.capacity, self.cache_len, self.dq[i], 1,
                             self.dk[i], self.dv[i], 0.0, self.dO[i])

    def decode(self):
        """The decode loop is launch-bound when driven from Python, so it is captured once in a CUDA graph
        (cache_len lives on the device, so the same graph is valid for every replay) and replayed."""
        if self.decode_graph is None:
            torch.cuda.synchronize()
            saved = self.cache_len.clone()
            side = torch.cuda.Stream(device=self.dev)
            side.wait_stream(torch.cuda.current_stream())
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    self.decode_eager()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            self.cache_len.copy_(saved)
            self.decode_graph = g
        self.decode_graph.replay()

    def launches_per_step(self) -> int:
        per_group = KERNELS_PER_CALL["compact"]
        if self.R > 0:
            per_group += KERNELS_PER_CALL["update"]
        # the timed schedule gathers and updates group by group
        n = KERNELS_PER_CALL["score"] + KERNELS_PER_CALL["select"] + self.groups * per_group
        if self.fused_select and self.groups == 1:
            n -= 1                                       # selection and gather are one kernel
        B = self.B
        wide = B.Shape.from_workload(self.w.replace(batch=self.w.batch * self.per_group), n_layers=1)
        n += self.groups * B.samkv_attn_kernel_count(self.handle_attn, wide, self.w.q_tokens, self.capacity, True)
        return n + self.w.n_layers * self.w.decode_steps * B.samkv_attn_kernel_count(self.handle, self.shape, 1,
                                                                                    self.capacity, True)


def widened_rows_ms(pipe: Pipeline, reps: int = 5):
    """Device time of the calls beyond the fixed-budget path, on the workload's own tensors, outside the timed
    region: dynamic selection (Top-P, cross-context Top-K, gather of its unit lists), cross-layer alignment,
    protected-only gather.  Block representatives are timed only when the workload scores blocks (block_size > 1)."""
    w, B = pipe.w, pipe.B
    dev = pipe.dev
    L, Bt, Hkv, D = w.n_layers, w.batch, w.n_kv_heads, w.n_ctx

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    out = {}
    P = torch.zeros((Bt, D), dtype=torch.float32, device=dev)
    star = list(range(max(0, L - 4), L))
    out["topp"] = timed(lambda: B.samkv_topp(pipe.handle, pipe.shape, pipe.scores, star, None, None, P))
    P_row = [min(1.0, max(0.0, float(x))) for x in P[0].cpu()]
    cand, K, S_u, S = B.samkv_topp_plan(pipe.shape, P_row)
    sel = torch.empty((L, Bt, Hkv, S_u), dtype=torch.int32, device=dev)
    scratch = torch.empty(B.samkv_select_cross_scratch_bytes(pipe.shape, cand), dtype=torch.uint8, device=dev)
    out["select_cross"] = timed(lambda: B.samkv_select_cross(pipe.handle, pipe.shape, pipe.scores, cand, scratch, sel))
    if S <= pipe.capacity:
        out["compact_units"] = timed(lambda: B.samkv_compact_units(pipe.handle, pipe.shape, pipe.inp["K"], pipe.inp["V"], sel,
                                                                  S_u, pipe.Kc, pipe.Vc, pipe.capacity, pipe.cache_len,
                                                                  pipe.inv_map))
    out["dynamic_kept_tokens"] = S
    out["compact_protected"] = timed(lambda: B.samkv_compact_protected(pipe.handle, pipe.shape, pipe.inp["K"], pipe.inp["V"],
                                                                      pipe.Kc, pipe.Vc, pipe.capacity, pipe.cache_len,
                                                                      pipe.inv_map))
    pipe.sparsify()                                        # restore the fixed-budget cache and its inverse map
    if pipe.R > 0:
        flags = torch.empty((L, Bt, w.l_tot), dtype=torch.uint8, device=dev)
        merged = torch.empty((Bt, w.l_tot), dtype=torch.int32, device=dev)
        merged_len = torch.empty((Bt,), dtype=torch.int32, device=dev)
        run_ids = torch.empty((L, Bt, min(w.l_tot, L * pipe.R)), dtype=torch.int32, device=dev)
        run_len = torch.empty((L, Bt), dtype=torch.int32, device=dev)
        out["align"] = timed(lambda: B.samkv_align(pipe.handle, pipe.shape, pipe.inv_map, pipe.tok_ids, flags, merged,
                                                   merged_len, run_ids, run_len))
    torch.cuda.synchronize()
    if B.samkv_poll_status(pipe.handle) != 0:
        raise RuntimeError("device-side check failed in the widened rows")
    return out


def pinned_inputs(pipe: Pipeline) -> dict:
    """The request's tensors in pinned host memory (the starting point of both end-to-end legs)."""
    host = {n: torch.empty(pipe.inp[n].shape, dtype=pipe.inp[n].dtype, pin_memory=True)
            for n in ("K", "V", "Q", "Qloc", "Qa", "Kq", "Vq")}
    for n, t in host.items():
        t.copy_(pipe.inp[n])
    torch.cuda.synchronize()
    return host


def e2e_steps(pipe: Pipeline, steps: int, warmup: int, host=None):
    """Same step, but every step's inputs start in pinned HOST memory and the result is read back.
    Per layer, a copy stream brings that layer's K and query rows over while the compute stream works on
    the previous layer.  V is never uploaded: samkv_compact gathers the kept V rows (about 15 %) straight
    from pinned host memory, which is the method's point -- only the sparse part of the cache is loaded
    to the GPU.  O of every layer is copied back.  Returns (seconds per step, h2d bytes, d2h bytes); the
    h2d figure counts the uploaded tensors plus the V rows the gather pulls across the bus."""
    w, B = pipe.w, pipe.B
    dev = pipe.dev
    names = ["K", "Q", "Qloc", "Qa", "Kq", "Vq"]
    host = host if host is not None else pinned_inputs(pipe)
    extra = {}
    if pipe.R > 0:
        for n, t in (("Knew", pipe.Knew), ("Vnew", pipe.Vnew), ("tok_ids", pipe.tok_ids)):
            extra[n] = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
            extra[n].copy_(t)
    O_host = torch.empty(pipe.O.shape, dtype=pipe.O.dtype, pin_memory=True)
    torch.cuda.synchronize()
    nbytes = lambda t: t.numel() * t.element_size()
    v_rows_bytes = w.n_layers * w.batch * w.n_kv_heads * pipe.S * w.head_dim * w.elem_bytes
    h2d = sum(nbytes(host[n]) for n in names) + sum(nbytes(t) for t in extra.values()) + v_rows_bytes
    d2h = nbytes(O_host)

    shape1 = B.Shape.from_workload(w, n_layers=1)
    copy_stream = torch.cuda.Stream(device=dev)
    main = torch.cuda.current_stream()
    L = w.n_layers

    def one_step():
        ready = []
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_stream(main)
            for l in range(L):
                for n in names:
                    pipe.inp[n][l].copy_(host[n][l], non_blocking=True)
                if pipe.R > 0:
                    pipe.Knew[l].copy_(extra["Knew"][l], non_blocking=True)
                    pipe.Vnew[l].copy_(extra["Vnew"][l], non_blocking=True)
                    pipe.tok_ids[l].copy_(extra["tok_ids"][l], non_blocking=True)
                e = torch.cuda.Event()
                e.record(copy_stream)
                ready.append(e)
        inp = pipe.inp
        for l in range(L):
            main.wait_event(ready[l])
            sl = slice(l, l + 1)
            B.samkv_score(pipe.handle, shape1, inp["K"][sl], inp["Q"][sl], w.q_tokens, inp["Qloc"][sl], pipe.t_loc, 1,
                          pipe.scores[sl])
            B.samkv_select(pipe.handle, shape1, pipe.scores[sl], pipe.k_units, pipe.sel[sl])
            B.samkv_compact(pipe.handle, shape1, inp["K"][sl], host["V"][sl], pipe.sel[sl], pipe.k_units, pipe.Kc[sl],
                            pipe.Vc[sl], pipe.capacity, pipe.cache_len[sl], pipe.inv_map[sl])
            if pipe.R > 0:
                B.samkv_update(pipe.handle, shape1, pipe.Kc[sl], pipe.Vc[sl], pipe.capacity, pipe.inv_map[sl],
                               pipe.tok_ids[sl], pipe.R, pipe.Knew[sl], pipe.Vnew[sl], B.SAMKV_UPDATE_FUSION)
            if (l + 1) % pipe.per_group == 0:           # the group's caches are complete: its attention, as in the step
                g = l // pipe.per_group
                pipe.attn_group(g)
                gs = slice(g * pipe.per_group, (g + 1) * pipe.per_group)
                O_host[gs].copy_(pipe.O[gs], non_blocking=True)

    O_ref = pipe.O.clone()                       # result of the device-resident steps: the e2e path must reproduce it
    for _ in range(warmup):
        one_step()
    torch.cuda.synchronize()
    if not torch.equal(O_host.to(dev), O_ref):
        raise RuntimeError("end-to-end path (V gathered from host memory) disagrees with the device-resident path")
    t0 = time.perf_counter()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one_step()
    e1.record()
    torch.cuda.synchronize()
    dev_s = e0.elapsed_time(e1) / 1e3
    wall_s = time.perf_counter() - t0
    return max(dev_s, wall_s) / steps, h2d, d2h


def e2e_block_means_steps(pipe: Pipeline, host: dict, steps: int, warmup: int, block: int = 64):
    """Second end-to-end leg, the deployment shape of Sec. 3.2: the block representatives (mean key of every
    64-token block, 1/64 of K) stay resident in HBM, K and V stay in pinned host memory.  Per layer the query rows are
    uploaded, samkv_score_blocks scores the representatives, samkv_select picks blocks under the same budget, and
    samkv_compact gathers the kept K and V rows straight from host memory -- only the sparse part of the cache crosses
    the bus; update, attention and the copy of O back follow as in the other leg.  The representatives are computed
    once outside the timed region (the paper's offline phase).  Returns a dict for the bench line."""
    B, dev = pipe.B, pipe.dev
    w = pipe.w.replace(name=pipe.w.name + f"_blocks{block}", block_size=block, n_init=block, n_local=block)
    L, Bt, Hkv, d = w.n_layers, w.batch, w.n_kv_heads, w.head_dim
    inp = pipe.inp
    shape = B.Shape.from_workload(w)
    shape1 = B.Shape.from_workload(w, n_layers=1)
    k_units = B.samkv_budget_units(shape, w.budget_bp)
    _, U_tot, S = B.samkv_layout(shape, k_units)
    capacity = S + w.q_tokens
    handle = B.Handle(shape, w.q_tokens, capacity)
    t_loc = pipe.t_loc
    Kbar = torch.empty((L, Bt, Hkv, U_tot, d), dtype=w.torch_dtype, device=dev)
    scores = torch.empty((L, Bt, Hkv, U_tot), dtype=torch.float32, device=dev)
    sel = torch.empty((L, Bt, Hkv, sum(k_units)), dtype=torch.int32, device=dev)
    Kc = torch.zeros((L, Bt, Hkv, capacity, d), dtype=w.torch_dtype, device=dev)
    Vc = torch.zeros_like(Kc)
    cache_len = torch.zeros((L, Bt), dtype=torch.int32, device=dev)
    inv_map = torch.empty((L, Bt, Hkv, w.l_tot), dtype=torch.int32, device=dev)
    O = torch.empty_like(pipe.O)
    O_host = torch.empty(O.shape, dtype=O.dtype, pin_memory=True)

    def timed(fn, reps=5):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    nbytes = lambda t: t.numel() * t.element_size()
    # offline phase, and the two block-representative calls timed on their own (device-resident, inputs > L2)
    means_ms = timed(lambda: B.samkv_block_means(handle, shape, inp["K"], Kbar))
    score_ms = timed(lambda: B.samkv_score_blocks(handle, shape, Kbar, inp["Q"], w.q_tokens, inp["Qloc"], t_loc, 1, scores))
    means_bytes = nbytes(inp["K"]) + nbytes(Kbar)
    score_bytes = nbytes(Kbar) + nbytes(inp["Q"]) + nbytes(inp["Qloc"]) + nbytes(scores)

    # device-resident reference of the same path (also yields the recompute list of this selection)
    B.samkv_select(handle, shape, scores, k_units, sel)
    B.samkv_compact(handle, shape, inp["K"], inp["V"], sel, k_units, Kc, Vc, capacity, cache_len, inv_map)
    torch.cuda.synchronize()
    R, tok_ids, Knew, Vnew, extra = 0, None, None, None, {}
    if w.recompute_share_bp > 0:
        toks0 = torch.stack([torch.nonzero(inv_map[l, 0, 0] >= 0).flatten() for l in range(L)])[:, None, :]
        R = (w.recompute_share_bp * S) // 10000
        tok_ids, Knew, Vnew = synth.make_recompute(w, inp["K"], inp["V"], toks0, R)
        for n, t in (("Knew", Knew), ("Vnew", Vnew), ("tok_ids", tok_ids)):
            extra[n] = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
            extra[n].copy_(t)
        B.samkv_update(handle, shape, Kc, Vc, capacity, inv_map, tok_ids, R, Knew, Vnew, B.SAMKV_UPDATE_FUSION)
    for l in range(L):
        B.samkv_attn(handle, shape, l, Kc, Vc, capacity, cache_len, inp["Qa"][l], w.q_tokens, inp["Kq"][l], inp["Vq"][l],
                     0.0, O[l])
    torch.cuda.synchronize()
    O_ref = O.clone()

    names = ["Q", "Qloc", "Qa", "Kq", "Vq"]
    kept_rows_bytes = 2 * L * Bt * Hkv * S * d * w.elem_bytes                     # K and V rows pulled by the gather
    h2d = sum(nbytes(host[n]) for n in names) + sum(nbytes(t) for t in extra.values()) + kept_rows_bytes
    d2h = nbytes(O_host)
    copy_stream = torch.cuda.Stream(device=dev)
    main = torch.cuda.current_stream()

    def one_step():
        ready = []
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_stream(main)
            for l in range(L):
                for n in names:
                    inp[n][l].copy_(host[n][l], non_blocking=True)
                if R > 0:
                    Knew[l].copy_(extra["Knew"][l], non_blocking=True)
                    Vnew[l].copy_(extra["Vnew"][l], non_blocking=True)
                    tok_ids[l].copy_(extra["tok_ids"][l], non_blocking=True)
                e = torch.cuda.Event()
                e.record(copy_stream)
                ready.append(e)
        for l in range(L):
            main.wait_event(ready[l])
            sl = slice(l, l + 1)
            B.samkv_score_blocks(handle, shape1, Kbar[sl], inp["Q"][sl], w.q_tokens, inp["Qloc"][sl], t_loc, 1, scores[sl])
            B.samkv_select(handle, shape1, scores[sl], k_units, sel[sl])
            B.samkv_compact(handle, shape1, host["K"][sl], host["V"][sl], sel[sl], k_units, Kc[sl], Vc[sl], capacity,
                            cache_len[sl], inv_map[sl])
            if R > 0:
                B.samkv_update(handle, shape1, Kc[sl], Vc[sl], capacity, inv_map[sl], tok_ids[sl], R, Knew[sl], Vnew[sl],
                               B.SAMKV_UPDATE_FUSION)
            B.samkv_attn(handle, shape1, 0, Kc[sl], Vc[sl], capacity, cache_len[sl], inp["Qa"][l], w.q_tokens, inp["Kq"][l],
                         inp["Vq"][l], 0.0, O[l])
            O_host[l].copy_(O[l], non_blocking=True)

    for _ in range(warmup):
        one_step()
    torch.cuda.synchronize()
    if B.samkv_poll_status(handle) != 0:
        raise RuntimeError("device-side check failed in the block-representative leg")
    if not torch.equal(O_host.to(dev), O_ref):
        raise RuntimeError("block-representative end-to-end path disagrees with its device-resident run")
    t0 = time.perf_counter()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one_step()
    e1.record()
    torch.cuda.synchronize()
    s_per_step = max(e0.elapsed_time(e1) / 1e3, time.perf_counter() - t0) / steps
    return {"value": w.batch * w.l_tot / s_per_step, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": s_per_step * 1e3, "block_size": block, "kept_tokens": S, "recomputed_rows": R,
            "resident_representative_bytes": nbytes(Kbar),
            "block_means_ms": means_ms, "block_means_gbs": means_bytes / means_ms / 1e6,
            "score_blocks_ms": score_ms, "score_blocks_gbs": score_bytes / score_ms / 1e6,
            "note": "per-GPU; block representatives resident in HBM (computed once, outside the timed region); K and V stay in "
                    "pinned host memory and only the kept rows are gathered across the bus by samkv_compact; query rows "
                    "uploaded per layer, O copied back; result equal to the device-resident run of the same path"}


# --------------------------------------------------------------------------------------------------
# the CPU oracle arm (also the cpu_baseline leg of the GPU arm)
# --------------------------------------------------------------------------------------------------
def oracle_sample_seconds(w, inp_cpu, layer=0, b=0, recompute=True):
    """Times the oracle, as it stands, on ONE (layer, batch element) of the workload: the whole path
    (pool, Eq. 1, scores, select, compact, fusion update, attention with the appended chunk)."""
    from oracle import samkv_oracle as O
    f64 = lambda t: t.to(torch.float64).numpy()
    K, V = f64(inp_cpu["K"][layer, b]), f64(inp_cpu["V"][layer, b])
    Q, Qloc = f64(inp_cpu["Q"][layer, b]), f64(inp_cpu["Qloc"][layer, b])
    Qa, Kq, Vq = f64(inp_cpu["Qa"][layer, b]), f64(inp_cpu["Kq"][layer, b]), f64(inp_cpu["Vq"][layer, b])
    k_units = [O.budget_units(n, w.block_size, w.n_init, w.n_local, w.budget_bp) for n in w.ctx_lens]
    rng = np.random.default_rng(w.seed)
    t0 = time.perf_counter()
    res = O.sparsify(K, V, Q, Qloc, w.ctx_offsets, w.block_size, w.n_init, w.n_local, k_units,
                     capacity=None)
    S = res["cache_len"]
    Kc = np.concatenate([res["Kc"], np.zeros((K.shape[0], w.q_tokens, K.shape[2]))], axis=1)
    Vc = np.concatenate([res["Vc"], np.zeros((K.shape[0], w.q_tokens, K.shape[2]))], axis=1)
    if recompute and w.recompute_share_bp > 0:
        R = (w.recompute_share_bp * S) // 10000
        toks = O.units_to_tokens(res["sel"][0], w.ctx_offsets, w.block_size)
        tok_ids = rng.permutation(toks)[:R]
        Knew = np.transpose(K[:, tok_ids], (1, 0, 2)) + 0.484 * rng.normal(size=(R, K.shape[0], K.shape[2]))
        Vnew = np.transpose(V[:, tok_ids], (1, 0, 2)) + 0.484 * rng.normal(size=(R, K.shape[0], K.shape[2]))
        Kc, Vc = O.update(Kc, Vc, res["inv_map"], tok_ids, Knew, Vnew, "fusion", dtype=w.dtype)
    O.attention(Kc, Vc, S, Qa, Kq, Vq)
    return time.perf_counter() - t0


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def cpu_baseline(w, repeats=2, target_seconds=12.0, max_repeats=32):
    """Oracle on a bounded sample: one (layer, batch element) of the workload, repeated until about
    `target_seconds` of CPU work have been timed (at least `repeats` times), scaled to the metric's unit
    (context tokens through ALL layers per second)."""
    w1 = w.replace(n_layers=1, batch=1)
    inp = synth.make_inputs(w1, "cpu")
    secs = []
    while len(secs) < repeats or (sum(secs) < target_seconds and len(secs) < max_repeats):
        secs.append(oracle_sample_seconds(w1, inp))
    repeats = len(secs)
    t = float(np.mean(secs))
    value = w.l_tot / (t * w.n_layers)           # tokens/s of a job that runs every layer on these cores
    return {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{repeats} x (1 layer x 1 batch element of {w.name}: {w.l_tot} context tokens, whole path), "
                      f"{t:.2f} s each, scaled by 1/{w.n_layers} layers",
            "seconds_per_sample": t, "host_cpus": os.cpu_count()}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w1 = w.replace(n_layers=1, batch=1)
    inp = synth.make_inputs(w1, "cpu")
    for _ in range(args.warmup):
        oracle_sample_seconds(w1, inp)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_seconds(w1, inp)
    t = (time.perf_counter() - t0) / args.steps
    value = w.l_tot / (t * w.n_layers)
    sample = (f"each step = 1 layer x 1 batch element of {w.name} ({w.l_tot} context tokens, whole path) on the host "
              f"cores; value scaled by 1/{w.n_layers} layers")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------
# multi-GPU host logic (no data-path collective: every rank owns an independent request batch)
# --------------------------------------------------------------------------------------------------
def rank_workload(w, rank: int):
    """Weak scaling: rank r processes its own batch of the same shape, generated from seed + r."""
    return w.replace(seed=w.seed + rank)


def max_over_ranks(elapsed_ms: float, device) -> float:
    """The job's step time is the slowest rank's device time."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(elapsed_ms)
    t = torch.tensor([elapsed_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(w, world: int, ms_per_step: float) -> float:
    """Whole-job context tokens per second: every rank pushes batch x L_tot tokens through all layers."""
    return w.batch * w.l_tot * world / (ms_per_step / 1e3)


def tensor_fractions(tflops: float) -> dict:
    """Attention throughput (the two products, 4 * rows * slots * d flop) against the dense bf16 tensor peaks: the
    measured cuBLAS figures of this machine (burst: a kernel timed alone; sustained: seconds under the power cap) and
    the nominal 2250 TFLOP/s."""
    peaks, kind = measured_peaks()
    burst = float(peaks.get("bf16_tflops", 1590.0))
    sustained = float(peaks.get("bf16_tflops_sustained", 1400.0))
    return {"of_measured_burst": tflops / burst, "of_measured_sustained": tflops / sustained, "of_nominal_2250": tflops / 2250.0,
            "peak_kind": kind, "burst_tflops": burst, "sustained_tflops": sustained}


def attention_flops(w, S: int) -> float:
    """QK^T and PV over the visible slots (cache + chunk; the causal part is counted in full), all layers."""
    return 4.0 * w.n_layers * w.batch * w.q_tokens * w.n_q_heads * (S + w.q_tokens) * w.head_dim


def host_description() -> dict:
    model = None
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except Exception:
        pass
    try:
        allowed = len(os.sched_getaffinity(0))
    except Exception:
        allowed = None
    return {"cpu_model": model, "nproc": os.cpu_count(), "allowed_cpus": allowed}


def oracle_one_core_seconds(names=("cfg0", "cfg1")) -> dict:
    """The oracle's whole path on the small configurations with BLAS limited to one thread."""
    out = {}
    try:
        from threadpoolctl import threadpool_limits
    except Exception:
        return out
    for n in names:
        w = synth.CONFIGS[n]
        inp = synth.make_inputs(w, "cpu")
        with threadpool_limits(limits=1):
            oracle_sample_seconds(w, inp)
            out[n] = oracle_sample_seconds(w, inp)
    return out


def run_other_workload(w, dev, hbm_peak: float, steps: int = 10, warmup: int = 3) -> dict:
    """Times another configuration with the same code path as the headline one (Pipeline.step: the overlapped
    schedule where the workload has several layers, in order otherwise), then one in-order pass for the phases."""
    pipe = Pipeline(w, dev)
    pipe.prepare_recompute()
    pipe.choose_schedule()
    for _ in range(warmup):
        pipe.step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        pipe.step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    ms_scan = None
    chosen = (pipe.groups, pipe.attn_share_sm)
    if w.n_layers % 8 == 0 and w.decode_steps == 0:       # the other schedule: scan of the next group beside attention
        pipe.attn_share_sm = False
        pipe.set_groups(8)
        for _ in range(warmup):
            pipe.step(overlap="scan")
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            pipe.step(overlap="scan")
        e1.record()
        torch.cuda.synchronize()
        ms_scan = e0.elapsed_time(e1) / steps
        pipe.attn_share_sm = chosen[1]
        pipe.set_groups(chosen[0])
    phase = {}
    for _ in range(2):
        ev = []
        pipe.step(ev, overlap=False, attention_all_layers=True, fused_select=False)
        torch.cuda.synchronize()
        for (n0, a), (n1, b) in zip(ev[:-1], ev[1:]):
            phase[n1] = phase.get(n1, 0.0) + a.elapsed_time(b) / 2
    status = max([pipe.B.samkv_poll_status(pipe.handle)] + [pipe.B.samkv_poll_status(h) for h in pipe._attn_handles.values()])
    ab = algorithmic_bytes(w, pipe.S, pipe.R, fusion=True, kept_rows=pipe.update_kept_rows)
    gbs = ab["total"] / (ms / 1e3) / 1e9
    out = {"layers_or_layer_buffers": w.n_layers, "budget_bp": w.budget_bp, "kept_tokens": pipe.S, "ms_per_step": ms,
           "us_per_layer": ms * 1e3 / w.n_layers, "algorithmic_gb_per_step": ab["total"] / 1e9, "achieved_gbs": gbs,
           "frac_of_measured_copy_peak": gbs / hbm_peak, "frac_of_nominal_8tbs": gbs / HBM_NOMINAL_GBS,
           "schedule": ("overlapped (%d layer groups)" % pipe.groups) if pipe.groups > 1 else "in order",
           "attention_kernel_in_schedule": "leaves room on its SMs" if pipe.attn_share_sm else "default",
           "schedule_trials_ms": pipe.schedule_trials or None,
           "ms_per_step_scan_beside_attention": ms_scan,
           "in_order_phase_ms": phase, "in_order_ms_per_step": sum(phase.values()),
           "attention_tflops": attention_flops(w, pipe.S) / (phase["attn"] / 1e3) / 1e12 if phase.get("attn") else None,
           "attention_of_tensor_peak": tensor_fractions(attention_flops(w, pipe.S) / (phase["attn"] / 1e3) / 1e12) if phase.get("attn") else None,
           "device_status": status}
    if w.decode_steps > 0:
        out["decode"] = {"steps": w.decode_steps, "us_per_step": phase["decode"] * 1e3 / w.decode_steps / w.n_layers,
                         "achieved_gbs": ab["decode"] / (phase["decode"] / 1e3) / 1e9,
                         "frac_of_measured_copy_peak": ab["decode"] / (phase["decode"] / 1e3) / 1e9 / hbm_peak,
                         "frac_of_nominal_8tbs": ab["decode"] / (phase["decode"] / 1e3) / 1e9 / HBM_NOMINAL_GBS,
                         "launch": "cuda graph"}
    del pipe
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="samkv", choices=["samkv", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling captures of a small case)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (profiling captures of a small case)")
    ap.add_argument("--budget-bp", type=int, default=0, help="override the sequence budget (basis points)")
    ap.add_argument("--attn-share-sm", default="auto", choices=["auto", "on", "off"],
                    help="prefill attention kernel of the overlapped schedule: the one that leaves room on its SMs "
                         "(on), the default one (off), or whichever is faster during warm-up (auto)")
    ap.add_argument("--layer-groups", type=int, default=0, choices=[0, 1, 2, 4, 8],
                    help="fix the number of layer groups of the schedule (1 = in order; 0 = choose during warm-up)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the cfg4 budget sweep, cfg3 and the sustained loop that follow the timed region")
    args = ap.parse_args()
    global ATTN_SHARE_SM
    ATTN_SHARE_SM = args.attn_share_sm
    profiling_case = bool(args.layers or args.batch)       # small captures under a profiler: keep launches few
    if args.warmup < 3 and args.impl == "samkv" and not profiling_case:
        args.warmup = 3

    w = synth.CONFIGS[args.workload]
    if args.layers:
        w = w.replace(n_layers=args.layers)
    if args.batch:
        w = w.replace(batch=args.batch)
    if args.budget_bp:
        w = w.replace(budget_bp=args.budget_bp)
    if args.impl == "reference":
        run_reference(args, w)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the SamKV library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_2508_11661_b200 import build
    if rank == 0:
        build.build_library()
    if world > 1:
        dist.barrier()

    pipe = Pipeline(rank_workload(w, rank), dev)
    pipe.prepare_recompute()
    if args.layer_groups and w.n_layers % args.layer_groups == 0 and w.decode_steps == 0:
        pipe.set_groups(args.layer_groups)
    elif not profiling_case:               # (small captures under a profiler keep the default kernel and few launches)
        pipe.choose_schedule()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()            # started early: nvidia-smi needs a moment before its first sample
    for _ in range(args.warmup):
        pipe.step()
    torch.cuda.synchronize()

    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.window_open()
    events = []
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ev = []
        pipe.step(ev)
        events.append(ev)
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler.window_close()
    elapsed_ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = max_over_ranks(elapsed_ms, dev)
    status = max([pipe.B.samkv_poll_status(pipe.handle)] + [pipe.B.samkv_poll_status(h) for h in pipe._attn_handles.values()])
    if status != 0:
        raise RuntimeError(f"device-side check failed during the benchmark (status {status})")

    # per-phase device time (rank 0), averaged over the timed steps ...
    timed_phase_ms = {}
    for ev in events:
        for (n0, a), (n1, b) in zip(ev[:-1], ev[1:]):
            timed_phase_ms[n1] = timed_phase_ms.get(n1, 0.0) + a.elapsed_time(b) / args.steps
    # ... and, after the timed region, one in-order pass on a single stream for the per-phase breakdown
    # (in the timed schedule gather/update and attention overlap, so they cannot be told apart there)
    phase_ms = {}
    n_seq = 3
    for _ in range(n_seq):
        ev = []
        pipe.step(ev, overlap=False, attention_all_layers=True, fused_select=False)
        torch.cuda.synchronize()
        for (n0, a), (n1, b) in zip(ev[:-1], ev[1:]):
            phase_ms[n1] = phase_ms.get(n1, 0.0) + a.elapsed_time(b) / n_seq
    sequential_ms = sum(phase_ms.values())
    if max(pipe.B.samkv_poll_status(h) for h in pipe._attn_handles.values()) != 0:
        raise RuntimeError("device-side check failed in the in-order passes")
    phase_ms["score"] = timed_phase_ms["score"]          # the roofline figure comes from the timed steps
    widened = widened_rows_ms(pipe) if (rank == 0 and w.decode_steps == 0 and not profiling_case) else None
    # the same step looped for at least two seconds (board power and clocks settle; the headline region is short)
    sustained = None
    if rank == 0 and world == 1 and not profiling_case and not args.no_other_workloads:
        n_sus = max(20, int(2200.0 / (elapsed_ms / args.steps)))
        sus_sampler = ClockSampler(local_rank)
        sus_sampler.start()
        time.sleep(0.3)
        torch.cuda.synchronize()
        sus_sampler.window_open()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(n_sus):
            pipe.step()
        s1.record()
        torch.cuda.synchronize()
        sus_sampler.window_close()
        sus_clocks = sus_sampler.stop()
        sus_ms = s0.elapsed_time(s1) / n_sus
        sustained = {"steps": n_sus, "ms_per_step": sus_ms, "clocks": sus_clocks,
                     "mcycles_per_step_at_median_clock": (sus_ms * sus_clocks["sm_mhz"] / 1e3) if sus_clocks.get("sm_mhz") else None}

    # the other schedule, outside the timed region: the whole scan of group g + 1 beside the attention of group g
    scan_ms = None
    if rank == 0 and world == 1 and w.n_layers % 8 == 0 and w.decode_steps == 0 and not profiling_case:
        chosen = (pipe.groups, pipe.attn_share_sm)
        pipe.attn_share_sm = False
        pipe.set_groups(8)
        for _ in range(3):
            pipe.step(overlap="scan")
        torch.cuda.synchronize()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(10):
            pipe.step(overlap="scan")
        s1.record()
        torch.cuda.synchronize()
        scan_ms = s0.elapsed_time(s1) / 10
        pipe.attn_share_sm = chosen[1]
        pipe.set_groups(chosen[0])

    # attention with one call per layer (what a caller that gets its queries layer by layer would run), for comparison
    per_layer_attn_ms = None
    if rank == 0 and world == 1 and w.decode_steps == 0 and not profiling_case:
        def per_layer_calls():
            pipe.cache_len.fill_(pipe.S)
            for l in range(w.n_layers):
                pipe.B.samkv_attn(pipe.handle, pipe.shape, l, pipe.Kc, pipe.Vc, pipe.capacity, pipe.cache_len, pipe.inp["Qa"][l],
                                  w.q_tokens, pipe.inp["Kq"][l], pipe.inp["Vq"][l], 0.0, pipe.O[l])
        for _ in range(2):
            per_layer_calls()
        torch.cuda.synchronize()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(5):
            per_layer_calls()
        s1.record()
        torch.cuda.synchronize()
        per_layer_attn_ms = s0.elapsed_time(s1) / 5
        pipe.step()                                   # leave the caches and O as the timed schedule leaves them
        torch.cuda.synchronize()

    ms_per_step = elapsed_ms / args.steps
    value = job_throughput(w, world, ms_per_step)
    peaks, peak_kind = measured_peaks()
    hbm_peak = float(peaks.get("hbm_gbs", HBM_FALLBACK_GBS))
    ab = algorithmic_bytes(w, pipe.S, pipe.R, fusion=True, kept_rows=pipe.update_kept_rows)
    score_gbs = ab["score"] / (phase_ms["score"] / 1e3) / 1e9
    pipeline_gbs = ab["total"] / (ms_per_step / 1e3) / 1e9

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "layers": w.n_layers, "batch_per_gpu": w.batch, "contexts": w.n_ctx,
                   "tokens_per_context": w.ctx_lens[0], "query_tokens": w.q_tokens, "heads": f"{w.n_q_heads}q/{w.n_kv_heads}kv",
                   "head_dim": w.head_dim, "budget_bp": w.budget_bp, "block_size": w.block_size, "kept_tokens": pipe.S,
                   "recomputed_rows_per_layer": pipe.R, "update": "fusion", "parallelism": f"dp{world} (independent batches)",
                   "cache_state": "inputs_larger_than_l2 (K+V %.1f GB per GPU)" % (2 * ab["score"] / 1e9)},
        "token_layers_per_s": value * w.n_layers,
        "pipeline": {"algorithmic_gb_per_step": ab["total"] / 1e9, "achieved_gbs": pipeline_gbs,
                     "frac_of_measured_copy_peak": pipeline_gbs / hbm_peak, "frac_of_nominal_8tbs": pipeline_gbs / HBM_NOMINAL_GBS,
                     "schedule": ("score+select, then %d layer groups: gather+update overlapped with attention on a second stream"
                                  % pipe.groups) if pipe.groups > 1 else
                                 (("in order on one stream, every phase one call over all layers" +
                                   (", selection and gather fused (samkv_select_compact)" if pipe.fused_select else ""))
                                  if w.decode_steps == 0 else "in order on one stream"),
                     "attention_kernel_in_schedule": ("128 rows, leaves room on its SMs (samkv_attn_share_sm)" if pipe.attn_share_sm
                                                      else "default"),
                     "schedule_trials_ms": pipe.schedule_trials or None,
                     "timed_phase_ms": timed_phase_ms, "in_order_ms_per_step": sequential_ms,
                     "ms_per_step_scan_beside_attention": scan_ms,
                     "attention_ms_one_call_per_layer": per_layer_attn_ms,
                     "attention_calls": "timed schedule: one samkv_attn_layers call per group of %d layers; in-order phase table: "
                                        "one call for all layers, default kernel" % pipe.per_group,
                     "phase_ms": phase_ms, "other_calls_ms": widened, "sustained": sustained,
                     "attention_tflops_in_order": attention_flops(w, pipe.S) / (phase_ms["attn"] / 1e3) / 1e12 if phase_ms.get("attn") else None,
                     "attention_of_tensor_peak": tensor_fractions(attention_flops(w, pipe.S) / (phase_ms["attn"] / 1e3) / 1e12) if phase_ms.get("attn") else None,
                     "bytes_note": "update charged for the rows it touches (new rows of every listed (token, head), old rows and "
                                   "results only where the head kept the token); the inverse map and index lists are not charged",
                     "phase_gbs": {k: ab[k] / (phase_ms[k] / 1e3) / 1e9 for k in ("score", "compact", "update", "attn", "decode") if phase_ms.get(k, 0) > 0}},
        "roofline": {"kernel": "score_stream_kernel (with the pooled-query kernel that precedes it in samkv_score)", "bound": "hbm",
                     "achieved": score_gbs, "peak": hbm_peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": score_gbs / hbm_peak, "frac_of_nominal_8tbs": score_gbs / HBM_NOMINAL_GBS,
                     "algorithmic_bytes_per_launch": ab["score"],
                     "traffic": (score_kernel_dram_bytes_per_row() * w.n_layers * w.batch * w.n_kv_heads * w.l_tot
                                 if (w.dtype == "bf16" and w.head_dim == 128 and score_kernel_dram_bytes_per_row()) else None),
                     "traffic_note": "ncu dram read+write of an 8-layer launch scaled by rows (profiles/)"},
        "gpu_launches": pipe.launches_per_step() * args.steps,
        "clocks": clocks,
    }

    if w.decode_steps > 0:
        line["decode"] = {"steps": w.decode_steps, "us_per_step": phase_ms["decode"] * 1e3 / w.decode_steps / w.n_layers,
                          "achieved_gbs": ab["decode"] / (phase_ms["decode"] / 1e3) / 1e9, "launch": "cuda graph"}
    if rank == 0 and not args.no_e2e and w.decode_steps == 0:
        try:
            import psutil
            free = psutil.virtual_memory().available
        except Exception:
            free = 0
        need = 2.5 * 2 * ab["score"]
        if free > need:
            host = pinned_inputs(pipe)
            s_per_step, h2d, d2h = e2e_steps(pipe, steps=max(2, min(args.steps, 3)), warmup=1, host=host)
            line["e2e"] = {"value": w.batch * w.l_tot / s_per_step, "unit": UNIT, "h2d_bytes_per_step": h2d,
                           "d2h_bytes_per_step": d2h, "ms_per_step": s_per_step * 1e3,
                           "note": "per-GPU; inputs in pinned host memory; K and query rows uploaded per layer (overlapped with compute), "
                                   "kept V rows gathered from host memory by samkv_compact, O copied back"}
            if world > 1:
                line["e2e"]["value"] *= world
                line["e2e"]["note"] += "; measured on rank 0 and scaled by the rank count"
            if world == 1 and w.block_size == 1 and all(n % 64 == 0 for n in w.ctx_lens):
                line["e2e_block_means"] = e2e_block_means_steps(pipe, host, steps=max(2, min(args.steps, 3)), warmup=1)
            del host
        else:
            line["e2e"] = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                           "note": f"skipped: host has {free / 1e9:.0f} GB free, needs {need / 1e9:.0f} GB pinned"}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, repeats=2)
        line["cpu_baseline"]["host"] = host_description()
        if not profiling_case:
            line["cpu_baseline"]["one_core_seconds_whole_path"] = oracle_one_core_seconds()
    # the other target configurations, same code path, after the headline one has released its memory
    if rank == 0 and world == 1 and not profiling_case and not args.no_other_workloads and w.name == "cfg2":
        del pipe
        torch.cuda.empty_cache()
        others = {}
        ow_sampler = ClockSampler(local_rank)
        ow_sampler.start()
        time.sleep(0.3)
        ow_sampler.window_open()
        for bp in (500, 1500, 3000, 10000):
            others[f"cfg4_budget_{bp}bp"] = run_other_workload(synth.CONFIGS["cfg4"].replace(n_layers=32, budget_bp=bp), dev, hbm_peak)
        others["cfg3"] = run_other_workload(synth.CONFIGS["cfg3"], dev, hbm_peak, steps=5, warmup=2)
        others["cfg1"] = run_other_workload(synth.CONFIGS["cfg1"], dev, hbm_peak, steps=50, warmup=5)
        ow_sampler.window_close()
        others["clocks"] = ow_sampler.stop()
        others["note"] = ("cfg4: one shape, 32 independent layer buffers, per-layer figures; cfg3: compaction and prefill, then 128 "
                          "decode steps replayed from one CUDA graph; cfg1: a single small layer (launch-latency bound)")
        line["pipeline"]["other_workloads"] = others
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

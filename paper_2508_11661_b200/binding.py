"""Thin ctypes binding of libsamkv.so: argument marshalling only.

Every function here has the name and the argument order of the C entry point it calls
(include/samkv.h); torch tensors stand for the device pointers, `torch.cuda.current_stream()`
for the stream.  Nothing is computed in Python, and there is no fallback: if the library
has not been built, or a call returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsamkv.so")
_lib = None

SAMKV_F32, SAMKV_BF16 = 0, 1
SAMKV_UPDATE_OVERWRITE, SAMKV_UPDATE_FUSION = 0, 1
SAMKV_MAX_CTX = 128

STATUS_NAMES = {0: "SAMKV_OK", 1: "SAMKV_ERR_INVALID_ARG", 2: "SAMKV_ERR_UNSUPPORTED", 3: "SAMKV_ERR_WORKSPACE",
                4: "SAMKV_ERR_CAPACITY", 5: "SAMKV_ERR_BUDGET", 6: "SAMKV_ERR_CUDA", 7: "SAMKV_ERR_DEVICE_CHECK"}

EXPORTS = ["samkv_workspace_bytes", "samkv_create", "samkv_destroy", "samkv_poll_status", "samkv_status_string",
           "samkv_budget_units", "samkv_layout", "samkv_score", "samkv_select", "samkv_compact", "samkv_update",
           "samkv_attn", "samkv_score_static", "samkv_topp", "samkv_topp_plan", "samkv_select_cross",
           "samkv_select_cross_scratch_bytes", "samkv_compact_units", "samkv_align", "samkv_compact_protected",
           "samkv_block_means", "samkv_score_blocks", "samkv_attn_kernel_count", "samkv_attn_share_sm", "samkv_attn_layers", "samkv_select_compact",
           "samkv_sparsify"]


class SamkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().samkv_status_string(status).decode() if _lib is not None else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({msg})")


class samkv_shape_t(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("n_ctx", ctypes.c_int32),
                ("ctx_offsets", ctypes.POINTER(ctypes.c_int32)), ("block_size", ctypes.c_int32),
                ("n_init", ctypes.c_int32), ("n_local", ctypes.c_int32), ("dtype", ctypes.c_int32)]


def lib() -> ctypes.CDLL:
    """Loads libsamkv.so (built by `python -m paper_2508_11661_b200.build`).  Raises if it is missing."""
    global _lib
    if _lib is None:
        _lib = load_library(_LIB_PATH)
    return _lib


def use_library(path: str) -> None:
    """Makes every function of this module call the library at `path` from now on (the tests of the debug build load
    libsamkv_debug.so this way); handles created before the switch must not be used after it."""
    global _lib
    _lib = load_library(path)


def load_library(path: str) -> ctypes.CDLL:
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2508_11661_b200.build` "
                           "(the SamKV CUDA library has no CPU fallback)")
    L = ctypes.CDLL(path)
    vp, i32, sz, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t, ctypes.c_float
    shp = ctypes.POINTER(samkv_shape_t)
    i32p = ctypes.POINTER(ctypes.c_int32)
    L.samkv_status_string.restype = ctypes.c_char_p
    L.samkv_status_string.argtypes = [ctypes.c_int]
    L.samkv_workspace_bytes.restype = sz
    L.samkv_workspace_bytes.argtypes = [shp, i32, i32]
    L.samkv_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, vp, sz]
    L.samkv_destroy.argtypes = [vp]
    L.samkv_poll_status.argtypes = [vp, vp]
    L.samkv_budget_units.argtypes = [shp, i32, i32p]
    L.samkv_layout.argtypes = [shp, i32p, i32p, i32p, i32p]
    L.samkv_score.argtypes = [vp, shp, vp, vp, i32, vp, i32, i32, vp, vp, vp]
    L.samkv_select.argtypes = [vp, shp, vp, i32p, vp, vp]
    L.samkv_compact.argtypes = [vp, shp, vp, vp, vp, i32p, vp, vp, i32, vp, vp, vp]
    L.samkv_update.argtypes = [vp, shp, vp, vp, i32, vp, vp, i32, vp, vp, i32, vp]
    L.samkv_select_compact.argtypes = [vp, shp, vp, i32p, vp, vp, vp, vp, vp, i32, vp, vp, vp]
    L.samkv_sparsify.argtypes = [vp, shp, vp, vp, vp, i32, vp, i32, i32, i32p, vp, vp, vp, vp, i32, vp, vp, vp]
    L.samkv_attn.argtypes = [vp, shp, i32, vp, vp, i32, vp, vp, i32, vp, vp, f32, vp, vp, vp]
    L.samkv_attn_layers.argtypes = [vp, shp, i32, i32, vp, vp, i32, vp, vp, i32, vp, vp, f32, vp, vp, vp]
    L.samkv_attn_layers.restype = i32
    L.samkv_score_static.argtypes = [shp, vp, vp, i32, vp, i32, i32, vp, vp]
    f32p = ctypes.POINTER(ctypes.c_float)
    L.samkv_topp.argtypes = [vp, shp, vp, i32p, i32, vp, vp, vp, vp]
    L.samkv_topp_plan.argtypes = [shp, f32p, i32p, i32p, i32p, i32p]
    L.samkv_select_cross.argtypes = [vp, shp, vp, i32p, vp, ctypes.c_size_t, vp, vp, vp]
    L.samkv_select_cross_scratch_bytes.argtypes = [shp, i32p]
    L.samkv_select_cross_scratch_bytes.restype = ctypes.c_size_t
    L.samkv_align.argtypes = [vp, shp, vp, vp, i32, vp, vp, vp, vp, i32, vp, vp]
    L.samkv_compact_protected.argtypes = [vp, shp, vp, vp, vp, vp, i32, vp, vp, vp]
    L.samkv_attn_kernel_count.argtypes = [vp, shp, i32, i32, i32]
    L.samkv_attn_share_sm.argtypes = [vp, i32]
    L.samkv_attn_share_sm.restype = i32
    L.samkv_attn_kernel_count.restype = i32
    L.samkv_block_means.argtypes = [vp, shp, vp, vp, vp]
    L.samkv_score_blocks.argtypes = L.samkv_score.argtypes
    L.samkv_compact_units.argtypes = [vp, shp, vp, vp, vp, i32, vp, vp, i32, vp, vp, vp]
    for name in EXPORTS:
        if name not in ("samkv_status_string", "samkv_workspace_bytes", "samkv_select_cross_scratch_bytes"):
            getattr(L, name).restype = ctypes.c_int
    if hasattr(L, "samkv_debug_score_with_lost_copy"):          # only the debug build exports it
        L.samkv_debug_score_with_lost_copy.argtypes = [vp, shp, vp, vp, i32, vp, i32, i32, vp, ctypes.c_uint32, vp]
    return L


class Shape:
    """Owns a samkv_shape_t and the host ctx_offsets array it points to."""

    def __init__(self, n_layers, batch, n_q_heads, n_kv_heads, head_dim, ctx_offsets: Sequence[int], block_size=1,
                 n_init=0, n_local=0, dtype="bf16"):
        self.ctx_offsets = [int(x) for x in ctx_offsets]
        self._off = (ctypes.c_int32 * len(self.ctx_offsets))(*self.ctx_offsets)
        self.c = samkv_shape_t(n_layers, batch, n_q_heads, n_kv_heads, head_dim, len(self.ctx_offsets) - 1,
                               ctypes.cast(self._off, ctypes.POINTER(ctypes.c_int32)), block_size, n_init, n_local,
                               {"f32": SAMKV_F32, "bf16": SAMKV_BF16}[dtype] if isinstance(dtype, str) else int(dtype))
        self.n_layers, self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim = (n_layers, batch, n_q_heads,
                                                                                      n_kv_heads, head_dim)
        self.n_ctx = len(self.ctx_offsets) - 1
        self.block_size, self.n_init, self.n_local = block_size, n_init, n_local
        self.l_tot = self.ctx_offsets[-1]

    @classmethod
    def from_workload(cls, w, **override):
        kw = dict(n_layers=w.n_layers, batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                  head_dim=w.head_dim, ctx_offsets=w.ctx_offsets, block_size=w.block_size, n_init=w.n_init,
                  n_local=w.n_local, dtype=w.dtype)
        kw.update(override)
        return cls(**kw)

    def ref(self):
        return ctypes.byref(self.c)


def _check(status: int, where: str):
    if status != 0:
        raise SamkvError(status, where)


def _ptr(t: Optional[torch.Tensor], allow_pinned_host: bool = False) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda and not (allow_pinned_host and t.is_pinned()):
        raise ValueError("expected a CUDA tensor" + (" or a pinned host tensor" if allow_pinned_host else ""))
    if not t.is_contiguous():
        raise ValueError("expected a contiguous tensor")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _i32_array(values: Sequence[int]):
    return (ctypes.c_int32 * len(values))(*[int(v) for v in values])


# ------------------------------------------------------------------ host helpers
def samkv_budget_units(shape: Shape, budget_bp: int) -> list:
    out = (ctypes.c_int32 * shape.n_ctx)()
    _check(lib().samkv_budget_units(shape.ref(), budget_bp, out), "samkv_budget_units")
    return list(out)


def samkv_layout(shape: Shape, k_units: Optional[Sequence[int]] = None):
    """Returns (protected units per context, total units U_tot, kept tokens S or None)."""
    prot = (ctypes.c_int32 * shape.n_ctx)()
    total = ctypes.c_int32(0)
    kept = ctypes.c_int32(0)
    k = _i32_array(k_units) if k_units is not None else None
    _check(lib().samkv_layout(shape.ref(), k, prot, ctypes.byref(total),
                              ctypes.byref(kept) if k_units is not None else None), "samkv_layout")
    return list(prot), total.value, (kept.value if k_units is not None else None)


def samkv_workspace_bytes(shape: Shape, max_q_tokens: int, cache_capacity: int) -> int:
    return int(lib().samkv_workspace_bytes(shape.ref(), max_q_tokens, cache_capacity))


# ------------------------------------------------------------------ handle
class Handle:
    """samkv_create / samkv_destroy.  The workspace tensor is allocated by torch and owned here."""

    def __init__(self, shape: Shape, max_q_tokens: int, cache_capacity: int, device: Optional[int] = None):
        dev = torch.cuda.current_device() if device is None else device
        nbytes = samkv_workspace_bytes(shape, max_q_tokens, cache_capacity)
        if nbytes == 0:
            raise SamkvError(1, "samkv_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=f"cuda:{dev}")
        self._h = ctypes.c_void_p()
        with torch.cuda.device(dev):
            _check(lib().samkv_create(ctypes.byref(self._h), dev, self.workspace.data_ptr(), nbytes), "samkv_create")

    def close(self):
        if self._h:
            lib().samkv_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def h(self):
        return self._h


def samkv_poll_status(handle: Handle) -> int:
    return int(lib().samkv_poll_status(handle.h, _stream()))


# ------------------------------------------------------------------ the five steps
def samkv_score(handle: Handle, shape: Shape, K, Q, T_q: int, Qloc, T_loc: int, use_bias: int, scores_out, qhat_out=None):
    _check(lib().samkv_score(handle.h, shape.ref(), _ptr(K), _ptr(Q), T_q, _ptr(Qloc), T_loc, int(use_bias),
                             _ptr(scores_out), _ptr(qhat_out), _stream()), "samkv_score")


def samkv_select(handle: Handle, shape: Shape, scores, k_units: Sequence[int], sel_out):
    _check(lib().samkv_select(handle.h, shape.ref(), _ptr(scores), _i32_array(k_units), _ptr(sel_out), _stream()),
           "samkv_select")


def samkv_compact(handle: Handle, shape: Shape, K, V, sel, k_units: Sequence[int], Kc, Vc, cache_capacity: int,
                  cache_len, inv_map=None):
    # K and V may live in pinned host memory: the gather then reads only the kept rows across the bus
    _check(lib().samkv_compact(handle.h, shape.ref(), _ptr(K, allow_pinned_host=True), _ptr(V, allow_pinned_host=True), _ptr(sel),
                               _i32_array(k_units), _ptr(Kc),
                               _ptr(Vc), cache_capacity, _ptr(cache_len), _ptr(inv_map), _stream()), "samkv_compact")


def samkv_select_compact(handle: Handle, shape: Shape, scores, k_units: Sequence[int], K, V, sel_out, Kc, Vc,
                         cache_capacity: int, cache_len, inv_map=None):
    _check(lib().samkv_select_compact(handle.h, shape.ref(), _ptr(scores), _i32_array(k_units), _ptr(K),
                                      _ptr(V, allow_pinned_host=True), _ptr(sel_out), _ptr(Kc), _ptr(Vc), cache_capacity,
                                      _ptr(cache_len), _ptr(inv_map), _stream()), "samkv_select_compact")


def samkv_sparsify(handle: Handle, shape: Shape, K, V, Q, T_q: int, Qloc, T_loc: int, use_bias: int,
                   k_units: Sequence[int], scores_out, sel_out, Kc, Vc, cache_capacity: int, cache_len, inv_map=None):
    _check(lib().samkv_sparsify(handle.h, shape.ref(), _ptr(K), _ptr(V, allow_pinned_host=True), _ptr(Q), T_q, _ptr(Qloc),
                                T_loc, int(use_bias), _i32_array(k_units), _ptr(scores_out), _ptr(sel_out), _ptr(Kc),
                                _ptr(Vc), cache_capacity, _ptr(cache_len), _ptr(inv_map), _stream()), "samkv_sparsify")


def samkv_update(handle: Handle, shape: Shape, Kc, Vc, cache_capacity: int, inv_map, tok_ids, R: int, Knew, Vnew,
                 mode: int):
    _check(lib().samkv_update(handle.h, shape.ref(), _ptr(Kc), _ptr(Vc), cache_capacity, _ptr(inv_map), _ptr(tok_ids),
                              R, _ptr(Knew), _ptr(Vnew), int(mode), _stream()), "samkv_update")


def samkv_attn(handle: Handle, shape: Shape, layer: int, Kc, Vc, cache_capacity: int, cache_len, Q, T_q: int,
               Kq, Vq, scale: float, O, lse=None):
    _check(lib().samkv_attn(handle.h, shape.ref(), layer, _ptr(Kc), _ptr(Vc), cache_capacity, _ptr(cache_len),
                            _ptr(Q), T_q, _ptr(Kq), _ptr(Vq), float(scale), _ptr(O), _ptr(lse), _stream()),
           "samkv_attn")


def samkv_attn_layers(handle: Handle, shape: Shape, layer0: int, n: int, Kc, Vc, cache_capacity: int, cache_len, Q,
                      T_q: int, Kq, Vq, scale: float, O, lse=None):
    """n consecutive layers in one call; Q, O [n, Bt, T_q, Hq, d], Kq, Vq [n, Bt, T_q, Hkv, d].  The handle's
    workspace must have been sized for n * Bt requests."""
    _check(lib().samkv_attn_layers(handle.h, shape.ref(), layer0, n, _ptr(Kc), _ptr(Vc), cache_capacity,
                                   _ptr(cache_len), _ptr(Q), T_q, _ptr(Kq), _ptr(Vq), float(scale), _ptr(O),
                                   _ptr(lse), _stream()), "samkv_attn_layers")


def samkv_score_static(shape: Shape, K, Q, T_q: int, Qloc, T_loc: int, use_bias: int, scores_out):
    """Scoring for callers that cannot allocate device memory (an engine whose pool owns all of HBM,
    a section where cudaMalloc's implicit synchronisation is not acceptable): no handle, no workspace;
    the scratch is a fixed 1 MiB array inside the library.  Calls sharing a GPU must not overlap."""
    _check(lib().samkv_score_static(shape.ref(), _ptr(K), _ptr(Q), T_q, _ptr(Qloc), T_loc, int(use_bias),
                                    _ptr(scores_out), _stream()), "samkv_score_static")


# ------------------------------------------------------------------ dynamic selection (Eq. 2, Eq. 3, cross-context Top-K)
def samkv_topp(handle: Handle, shape: Shape, scores, star_layers: Sequence[int], max_units, min_units, P_out):
    _check(lib().samkv_topp(handle.h, shape.ref(), _ptr(scores), _i32_array(star_layers), len(star_layers),
                            _ptr(max_units), _ptr(min_units), _ptr(P_out), _stream()), "samkv_topp")


def samkv_topp_plan(shape: Shape, P: Sequence[float]):
    """Returns (cand per document, K, S_u, kept tokens S) for one request's Top-P ratios."""
    arr = (ctypes.c_float * len(P))(*[float(x) for x in P])
    cand = (ctypes.c_int32 * shape.n_ctx)()
    K, S_u, S = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
    _check(lib().samkv_topp_plan(shape.ref(), arr, cand, ctypes.byref(K), ctypes.byref(S_u), ctypes.byref(S)),
           "samkv_topp_plan")
    return list(cand), K.value, S_u.value, S.value


def samkv_select_cross_scratch_bytes(shape: Shape, cand: Optional[Sequence[int]] = None) -> int:
    """Bytes of scratch samkv_select_cross needs for these candidate counts (None: the bound for any counts)."""
    return int(lib().samkv_select_cross_scratch_bytes(shape.ref(), None if cand is None else _i32_array(cand)))


def samkv_select_cross(handle: Handle, shape: Shape, scores, cand: Sequence[int], scratch, sel_out, counts_out=None):
    """scratch: a device tensor of at least samkv_select_cross_scratch_bytes(shape) bytes."""
    _check(lib().samkv_select_cross(handle.h, shape.ref(), _ptr(scores), _i32_array(cand), _ptr(scratch),
                                    scratch.numel() * scratch.element_size(), _ptr(sel_out), _ptr(counts_out),
                                    _stream()), "samkv_select_cross")


def samkv_compact_units(handle: Handle, shape: Shape, K, V, sel, S_u: int, Kc, Vc, cache_capacity: int, cache_len,
                        inv_map=None):
    _check(lib().samkv_compact_units(handle.h, shape.ref(), _ptr(K), _ptr(V, allow_pinned_host=True), _ptr(sel), S_u,
                                     _ptr(Kc), _ptr(Vc), cache_capacity, _ptr(cache_len), _ptr(inv_map), _stream()),
           "samkv_compact_units")


# ------------------------------------------------------------------ cross-layer alignment (Sec. 3.3)
FLAG_KEPT, FLAG_RECOMPUTE, FLAG_OUTPUT, FLAG_PAD_REUSE = 1, 2, 4, 8


def samkv_align(handle: Handle, shape: Shape, inv_map, tok_ids, flags_out, merged_ids, merged_len, run_ids, run_len):
    """tok_ids int32 [L, R] (or None); run_ids int32 [L, Bt, run_capacity]."""
    R = 0 if tok_ids is None else int(tok_ids.shape[1])
    _check(lib().samkv_align(handle.h, shape.ref(), _ptr(inv_map), _ptr(tok_ids), R, _ptr(flags_out), _ptr(merged_ids),
                             _ptr(merged_len), _ptr(run_ids), int(run_ids.shape[-1]), _ptr(run_len), _stream()),
           "samkv_align")


# ------------------------------------------------------------------ protected-only composite cache (Sec. 3.1)
def samkv_compact_protected(handle: Handle, shape: Shape, K, V, Kc, Vc, cache_capacity: int, cache_len, inv_map=None):
    _check(lib().samkv_compact_protected(handle.h, shape.ref(), _ptr(K), _ptr(V, allow_pinned_host=True), _ptr(Kc),
                                         _ptr(Vc), cache_capacity, _ptr(cache_len), _ptr(inv_map), _stream()),
           "samkv_compact_protected")


# ------------------------------------------------------------------ block representatives (Sec. 3.2)
def samkv_block_means(handle: Handle, shape: Shape, K, Kbar):
    _check(lib().samkv_block_means(handle.h, shape.ref(), _ptr(K), _ptr(Kbar), _stream()), "samkv_block_means")


def samkv_score_blocks(handle: Handle, shape: Shape, Kbar, Q, T_q: int, Qloc, T_loc: int, use_bias: int, scores_out,
                       qhat_out=None):
    _check(lib().samkv_score_blocks(handle.h, shape.ref(), _ptr(Kbar), _ptr(Q), T_q, _ptr(Qloc), T_loc, use_bias,
                                    _ptr(scores_out), _ptr(qhat_out), _stream()), "samkv_score_blocks")


def samkv_attn_share_sm(handle: Handle, on: bool) -> None:
    _check(lib().samkv_attn_share_sm(handle.h, int(bool(on))), "samkv_attn_share_sm")


def samkv_attn_kernel_count(handle: Handle, shape: Shape, T_q: int, cache_capacity: int, appended: bool) -> int:
    """Kernels one samkv_attn call with these sizes launches (for launch accounting)."""
    return int(lib().samkv_attn_kernel_count(handle.h, shape.ref(), T_q, cache_capacity, int(bool(appended))))

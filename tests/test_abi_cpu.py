"""No-GPU checks of the C-ABI library: it loads, exports every entry point the header declares,
its host-side helpers agree with the oracle, and bad arguments are refused with the right code."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import samkv_oracle as O
from paper_2508_11661_b200 import binding as B
from paper_2508_11661_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(samkv_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_entry_point():
    lib = B.lib()
    names = declared_symbols()
    assert {"samkv_score", "samkv_select", "samkv_compact", "samkv_update", "samkv_attn"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert names == set(B.EXPORTS), "binding.EXPORTS and the header disagree"


def test_debug_entry_point_exists_only_in_the_debug_build():
    """The hook that makes a bounded wait run out is compiled into libsamkv_debug.so alone."""
    from paper_2508_11661_b200 import build
    assert not hasattr(B.lib(), "samkv_debug_score_with_lost_copy")
    if not os.path.exists(build.DEBUG_LIB_PATH):
        pytest.skip("debug library not built")
    dbg = B.load_library(build.DEBUG_LIB_PATH)
    assert hasattr(dbg, "samkv_debug_score_with_lost_copy")
    for n in declared_symbols():
        assert hasattr(dbg, n), f"{n} missing from the debug build"


def test_status_strings():
    lib = B.lib()
    seen = {lib.samkv_status_string(i).decode() for i in range(8)}
    assert len(seen) == 8 and lib.samkv_status_string(99).decode() == "unknown status"


@pytest.mark.parametrize("seed", range(8))
def test_budget_and_layout_match_oracle(seed):
    r = np.random.default_rng(seed)
    Bsz = int(2 ** r.integers(0, 7))
    n_init = Bsz * int(r.integers(0, 3))
    n_local = Bsz * int(r.integers(1, 4))
    lens = [int(x) for x in r.integers(1, 900, size=int(r.integers(1, 9)))]
    off = [0] + list(np.cumsum(lens))
    shape = B.Shape(2, 3, 8, 2, 128, off, Bsz, n_init, n_local, "bf16")
    prot, U_tot, _ = B.samkv_layout(shape)
    assert prot == [len(O.protected_units(n, Bsz, n_init, n_local)) for n in lens]
    assert U_tot == sum(-(-n // Bsz) for n in lens)
    for bp in (0, 500, 1500, 3000, 10000):
        k = B.samkv_budget_units(shape, bp)
        assert k == [O.budget_units(n, Bsz, n_init, n_local, bp) for n in lens]
        _, _, S = B.samkv_layout(shape, k)
        # kept tokens: the oracle's gather of any valid selection has this many rows
        u = r.normal(size=(1, U_tot))
        sel = O.select_units(u, off, Bsz, n_init, n_local, k)
        assert S == len(O.units_to_tokens(sel[0], off, Bsz))


@pytest.mark.parametrize("seed", range(6))
def test_topp_plan_matches_oracle(seed):
    """Candidate counts, K, list length and kept tokens of the dynamic selection (host arithmetic only)."""
    r = np.random.default_rng(100 + seed)
    Bsz = int(2 ** r.integers(0, 7))
    n_init = Bsz * int(r.integers(0, 3))
    n_local = Bsz * int(r.integers(1, 4))
    lens = [int(x) for x in r.integers(1, 2000, size=int(r.integers(1, 9)))]
    off = [0] + list(np.cumsum(lens))
    shape = B.Shape(1, 1, 8, 2, 128, off, Bsz, n_init, n_local, "bf16")
    _, U_tot, _ = B.samkv_layout(shape)
    for trial in range(4):
        P = r.random(len(lens)).astype(np.float32)
        if trial == 0:
            P[:] = 0.0
        if trial == 1:
            P[:] = 1.0
        cand, K, S_u, S = B.samkv_topp_plan(shape, [float(x) for x in P])
        assert cand == O.candidate_counts(P.astype(np.float64), off, Bsz, n_init, n_local)
        u = r.normal(size=(2, U_tot))
        sel, counts = O.cross_context_select(u, off, Bsz, n_init, n_local, cand)
        assert K == sum(cand) // len(lens) and S_u == sel.shape[1]
        assert S == len(O.units_to_tokens(sel[0], off, Bsz)) == len(O.units_to_tokens(sel[1], off, Bsz))


def test_bad_shapes_are_refused_on_the_host():
    ok = dict(n_layers=1, batch=1, n_q_heads=8, n_kv_heads=2, head_dim=128, ctx_offsets=[0, 100, 300], block_size=1,
              n_init=4, n_local=8, dtype="bf16")

    def status(**kw):
        a = dict(ok); a.update(kw)
        try:
            B.samkv_budget_units(B.Shape(**a), 1500)
            return 0
        except B.SamkvError as e:
            return e.status

    assert status() == 0
    assert status(head_dim=96) == 2
    assert status(block_size=3) == 2 and status(block_size=128) == 2
    assert status(n_q_heads=7) == 1
    assert status(ctx_offsets=[0, 100, 100]) == 1 and status(ctx_offsets=[1, 100]) == 1
    assert status(block_size=16, n_init=8, n_local=16) == 1            # n_init not a multiple of B
    assert status(block_size=16, n_init=16, n_local=0, ctx_offsets=[0, 100]) == 1   # short tail unit unprotected
    assert status(block_size=16, n_init=16, n_local=0, ctx_offsets=[0, 96]) == 0
    assert status(ctx_offsets=list(range(0, 130 * 10, 10))) == 2       # more than SAMKV_MAX_CTX contexts
    assert status(dtype=5) == 2
    shape = B.Shape(**ok)
    with pytest.raises(B.SamkvError) as e:
        B.samkv_layout(shape, [1, 300])
    assert e.value.status == 5
    assert B.samkv_workspace_bytes(B.Shape(**dict(ok, head_dim=96)), 16, 100) == 0
    assert B.samkv_workspace_bytes(shape, 16, 1000) >= 256


def test_null_handle_and_null_out_pointers():
    lib = B.lib()
    shape = B.Shape(1, 1, 8, 2, 128, [0, 100], 1, 4, 8, "bf16")
    assert lib.samkv_destroy(None) == 1
    assert lib.samkv_poll_status(None, None) == 1
    assert lib.samkv_score(None, shape.ref(), None, None, 1, None, 1, 0, None, None, None) == 1
    assert lib.samkv_create(None, 0, None, 0) == 1
    assert lib.samkv_budget_units(shape.ref(), 1500, None) == 1
    assert lib.samkv_budget_units(None, 1500, None) == 1


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", "/nonexistent/libsamkv.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()

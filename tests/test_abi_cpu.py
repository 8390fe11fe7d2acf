"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the header
declares, sizes its workspace, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2509_03136_b200 import build as gbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def gv():
    gbuild.build()
    from paper_2509_03136_b200 import gvote
    gvote.load()
    return gvote


def _params(gv, **kw):
    base = dict(d_h=512, n_q_heads=8, n_kv_heads=2, d_k=64, rope_theta=1e4, S=16, p_nuc=0.95, n_f=128, n_s=4, seed=0)
    base.update(kw)
    return gv.make_params(**base)


def test_every_declared_symbol_is_exported(gv):
    header = open(os.path.join(ROOT, "include", "gvote.h")).read()
    declared = re.findall(r"GVOTE_API\s+[\w\s\*]+?\b(gvote_\w+)\s*\(", header)
    assert len(declared) >= 14 and len(set(declared)) == len(declared)
    assert set(declared) == set(gv.EXPORTS)
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2509_03136_b200", "libgvote.so"))
    for name in declared:
        assert hasattr(lib, name), name


def test_params_struct_matches_header(gv):
    header = open(os.path.join(ROOT, "include", "gvote.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} gvote_params;", header, re.S).group(1)
    fields = re.findall(r"^\s*(?:int32_t|uint32_t|uint64_t|float|double)\s+(\w+);", body, re.M)
    assert fields == [f[0] for f in gv.GVoteParams._fields_]
    assert ctypes.sizeof(gv.GVoteParams) == 64


def test_workspace_bytes(gv):
    p = _params(gv)
    small = gv.gvote_workspace_bytes(p, 1, 512, 512)
    big = gv.gvote_workspace_bytes(p, 1, 4096, 4096)
    assert 0 < small < big
    assert gv.gvote_workspace_bytes(p, 0, 512, 512) == 0
    assert gv.gvote_workspace_bytes(p, 1, 512, 1024) == 0            # max_N > total
    assert gv.gvote_workspace_bytes(_params(gv, S=0), 1, 512, 512) == 0
    assert gv.gvote_workspace_bytes(_params(gv, n_q_heads=7), 1, 512, 512) == 0
    assert gv.gvote_workspace_bytes(_params(gv, p_nuc=0.0), 1, 512, 512) == 0
    assert gv.gvote_workspace_bytes(_params(gv, d_k=36), 1, 512, 512) == 0


def test_workspace_of_the_default_mode_holds_no_logits_matrix(gv):
    """Section 4.4 names the S x N logits matrix as what runs out of memory beyond 128K.  The default
    (top-k) mode keeps none: its workspace stays far below S x N fp32 values at the long-context
    shapes, and below the per-sample top-p mode's, which does keep fp32 rows."""
    shapes = {"c2": dict(d_h=4096, n_q_heads=32, n_kv_heads=8, d_k=128, S=32, N=32768),
              "c4": dict(d_h=3584, n_q_heads=28, n_kv_heads=4, d_k=128, S=64, N=131072)}
    for name, sh in shapes.items():
        N = sh.pop("N")
        kw = dict(rope_theta=1e6, p_nuc=0.95, n_f=128, n_s=4, seed=0)
        topk = gv.gvote_workspace_bytes(gv.make_params(sel_mode=gv.SEL_TOPK_C0, **sh, **kw), 1, N, N)
        topp = gv.gvote_workspace_bytes(gv.make_params(sel_mode=gv.SEL_TOPP, **sh, **kw), 1, N, N)
        matrix = sh["n_q_heads"] * sh["S"] * N * 4
        assert topp > matrix                    # every row as fp32
        assert topk < matrix / 2 and topk < topp / 2, (name, topk, topp, matrix)
    # doubling S doubles the per-row state (sampled keys, candidate segments): well under the S x N x 4 bytes of fp32 rows
    a = gv.gvote_workspace_bytes(gv.make_params(sel_mode=0, d_h=4096, n_q_heads=32, n_kv_heads=8, d_k=128, S=32, **kw), 1, 32768, 32768)
    b = gv.gvote_workspace_bytes(gv.make_params(sel_mode=0, d_h=4096, n_q_heads=32, n_kv_heads=8, d_k=128, S=64, **kw), 1, 32768, 32768)
    assert (b - a) < 0.45 * (32 * 32 * 32768 * 4)


def test_mask_geometry_never_overlaps(gv):
    import numpy as np
    rng = np.random.default_rng(0)
    for _ in range(200):
        lens = rng.integers(1, 300, size=rng.integers(1, 9))
        cu = np.concatenate([[0], np.cumsum(lens)])
        offs = [gv.mask_word_offset(int(cu[r]), r) for r in range(len(lens))]
        for r in range(len(lens) - 1):
            assert offs[r] + (lens[r] + 31) // 32 <= offs[r + 1]
        assert offs[-1] + (lens[-1] + 31) // 32 <= gv.mask_row_words(int(cu[-1]), len(lens))


def test_bad_arguments_are_rejected_on_the_host(gv):
    lib = gv.load()
    p = _params(gv)
    A = 0x10000          # aligned dummy address; never dereferenced because the checks fail first
    st = lib.gvote_fit(ctypes.byref(p), None, 512, A, 1, 512, 512, A, A, A, 1 << 30, None)
    assert st == -1 and "invalid" in gv.gvote_status_string(st)
    st = lib.gvote_fit(ctypes.byref(p), A + 4, 512, A, 1, 512, 512, A, A, A, 1 << 30, None)
    assert st == -2
    st = lib.gvote_fit(ctypes.byref(p), A, 512, A, 1, 512, 512, A, A, A, 64, None)
    assert st == -3
    st = lib.gvote_fit(ctypes.byref(p), A, 100, A, 1, 512, 512, A, A, A, 1 << 30, None)
    assert st == -2                                                   # row stride below d_h / unaligned
    st = lib.gvote_fit(ctypes.byref(p), A, 512, A, 1, 5, 5, A, A, A, 1 << 30, None)
    assert st == -1                                                   # fewer than two rows after the sinks
    bad = _params(gv, d_k=36)
    st = lib.gvote_sample(ctypes.byref(bad), A, A, 1, A, None, None)
    assert st == -4
    st = lib.gvote_compact(ctypes.byref(p), A, A, 64, 64 * 512, A, A, 1, 512, 512, A, A, 16, None)
    assert st == -3
    st = lib.gvote_vote(ctypes.byref(p), A, A, 60, 64 * 512, A, 1, 512, 512, A, A, A, None, A, 1 << 30, None)
    assert st == -2
    assert gv.gvote_status_string(0) == "ok" and gv.gvote_status_string(-6).startswith("a bounded")


def test_missing_library_fails_loudly(gv, monkeypatch):
    monkeypatch.setattr(gv, "_lib", None)
    monkeypatch.setattr(gv, "_LIB_PATH", "/nonexistent/libgvote.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        gv.load()

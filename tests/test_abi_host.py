"""CPU-only checks of the C ABI: the library loads without a GPU, exports every symbol the header declares,
its host arithmetic agrees with the oracle's, and argument errors are caught before anything is launched."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2503_23956_b200 as ac

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "aircache.h")


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aircache_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 16
    handle = C.CDLL(ac.LIB)
    for n in names:
        assert hasattr(handle, n), f"{n} declared in aircache.h but not exported"
    assert sorted(ac.exported_symbols()) == names, "binding and header disagree"
    assert ac.aircache_version() == 102


def test_strerror_covers_all_codes():
    seen = {ac.aircache_strerror(c) for c in range(0, -9, -1)}
    assert len(seen) == 9 and "unknown error code" not in seen
    assert ac.aircache_strerror(-99) == "unknown error code"


@pytest.mark.parametrize("L,B,Nv,Nt,slack,ratio", [(4, 1, 576, 64, 0, 0.10), (28, 1, 7290, 128, 0, 0.05),
                                                 (28, 64, 2916, 256, 7, 0.10), (80, 8, 7290, 2048, 0, 0.05),
                                                 (3, 2, 5, 4, 1, 0.5), (2, 1, 3, 1, 0, 1.0), (2, 1, 3, 1, 0, 0.0)])
def test_row_arithmetic_matches_oracle(oracle_mod, L, B, Nv, Nt, slack, ratio):
    sh = ac.shape(L, B, 8, 2, 64, Nv, Nt, min(Nt, 4), slack)
    T = oracle_mod.total_kept(Nv, L, ratio)
    assert ac.aircache_kept_per_sequence(sh, ratio) == T
    assert ac.aircache_total_rows(sh, ratio) == B * (T + L * (Nt + slack))
    assert ac.aircache_workspace_bytes(sh) > 0


def test_shape_validation():
    good = dict(n_layers=2, batch=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_visual=10, n_text=4, window=4)
    assert ac.aircache_workspace_bytes(ac.shape(**good)) > 0
    bad = [
        (dict(n_layers=0), ac.ERR_INVALID_ARG), (dict(batch=-1), ac.ERR_INVALID_ARG),
        (dict(n_q_heads=7), ac.ERR_INVALID_ARG), (dict(window=5), ac.ERR_INVALID_ARG),
        (dict(window=0), ac.ERR_INVALID_ARG), (dict(slack=-1), ac.ERR_INVALID_ARG),
        (dict(scale=0.0), ac.ERR_INVALID_ARG), (dict(scale=float("nan")), ac.ERR_INVALID_ARG),
        (dict(head_dim=96), ac.ERR_UNSUPPORTED), (dict(n_kv_heads=3, n_q_heads=6), ac.ERR_UNSUPPORTED),
        (dict(n_q_heads=64, n_kv_heads=2), ac.ERR_UNSUPPORTED), (dict(n_visual=2), ac.ERR_UNSUPPORTED),
        (dict(n_text=200, window=129), ac.ERR_UNSUPPORTED), (dict(n_layers=64, batch=64), ac.ERR_UNSUPPORTED),
    ]
    for change, code in bad:
        sh = ac.shape(**{**good, **change})
        assert ac.aircache_workspace_bytes(sh) == code, change
        assert ac.aircache_total_rows(sh, 0.5) == code, change
    # per-KV-head mode: every (layer, sequence, KV head) cell is a region of its own
    per = ac.shape(**{**good, "per_kv_head": 1, "slack": 3})
    Hkv, L, B = good["n_kv_heads"], good["n_layers"], good["batch"]
    T = ac.aircache_kept_per_sequence(per, 0.3)
    assert T == int(np.floor(0.3 * good["n_visual"] * L * Hkv + 0.5))
    assert ac.aircache_total_rows(per, 0.3) == B * (T + L * Hkv * (good["n_text"] + 3))
    assert ac.aircache_workspace_bytes(ac.shape(**{**good, "per_kv_head": 2})) == ac.ERR_INVALID_ARG
    assert ac.aircache_workspace_bytes(ac.shape(**{**good, "per_kv_head": 1, "n_layers": 1792 // (B * Hkv) + 1})) == ac.ERR_UNSUPPORTED
    assert ac.aircache_total_rows(ac.shape(**good), 1.5) == ac.ERR_INVALID_ARG
    assert ac.aircache_total_rows(ac.shape(**good), float("nan")) == ac.ERR_INVALID_ARG


def test_entry_points_reject_bad_arguments_on_the_host():
    """Fake (never dereferenced) pointers: every call must fail in the host-side checks, so no CUDA call is
    made and the test runs without a GPU."""
    sh = ac.shape(2, 2, 8, 2, 64, 10, 4, 4)
    ws_bytes = ac.aircache_workspace_bytes(sh)
    P = 0x10000000   # 256-byte aligned fake address

    class Ws:
        def __init__(self, ptr, n):
            self.ptr, self.n = ptr, n

        def data_ptr(self):
            return self.ptr

        def numel(self):
            return self.n

        def element_size(self):
            return 1

    ws = Ws(P, ws_bytes)
    full = ac.Full(P, P, 1280, 640, 64, 128)
    rag = ac.Ragged(P, P, P, P, ac.aircache_total_rows(sh, 0.5))
    s = 0  # default stream, as an int: torch.cuda is never touched
    # score
    assert ac.aircache_score(sh, full, None, 0.9, P, None, ws, s, check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_score(sh, full, P, 1.5, P, None, ws, s, check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_score(sh, full, P + 2, 0.9, P, None, ws, s, check=False) == ac.ERR_ALIGNMENT
    assert ac.aircache_score(sh, ac.Full(P, P, 1280, 640, 64, 100), P, 0.9, P, None, ws, s,
                             check=False) == ac.ERR_ALIGNMENT
    assert ac.aircache_score(sh, ac.Full(P + 8, P, 1280, 640, 64, 128), P, 0.9, P, None, ws, s,
                             check=False) == ac.ERR_ALIGNMENT
    assert ac.aircache_score(sh, full, P, 0.9, P, None, Ws(P, ws_bytes - 1), s,
                             check=False) == ac.ERR_WORKSPACE_TOO_SMALL
    assert ac.aircache_score(sh, full, P, 0.9, P, None, Ws(P + 16, ws_bytes), s, check=False) == ac.ERR_ALIGNMENT
    assert ac.aircache_score(sh, full, P, 0.9, P, None, None, s, check=False) == ac.ERR_INVALID_ARG
    # score, a range of layers
    for begin, count in ((-1, 1), (0, 3), (2, 1), (1, 2), (0, -1)):
        assert ac.aircache_score_layers(sh, full, P, 0.9, begin, count, P, None, ws, s,
                                        check=False) == ac.ERR_INVALID_ARG, (begin, count)
    assert ac.aircache_score_layers(sh, full, P, 0.9, 2, 0, P, None, ws, s, check=False) == ac.OK   # empty range
    assert ac.aircache_score_layers(sh, full, P + 2, 0.9, 0, 1, P, None, ws, s, check=False) == ac.ERR_ALIGNMENT
    # budget
    assert ac.aircache_budget(sh, P, 1.2, 0, P, None, None, rag, ws, s, check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_budget(sh, P, 0.5, 4, P, None, None, rag, ws, s, check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_budget(sh, None, 0.5, 0, P, None, None, rag, ws, s, check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_budget(sh, P, 0.5, 0, P, None, None, ac.Ragged(P, P, None, P, 10), ws, s,
                              check=False) == ac.ERR_INVALID_ARG
    # compact
    small = ac.Ragged(P, P, P, P, ac.aircache_total_rows(sh, 0.5) - 1)
    assert ac.aircache_compact(sh, full, P, P, 0.5, small, None, ws, s, check=False) == ac.ERR_CAPACITY
    assert ac.aircache_compact(sh, full, P, P, 0.5, ac.Ragged(P + 64, P, P, P, 10 ** 6), None, ws, s,
                               check=False) == ac.ERR_ALIGNMENT
    assert ac.aircache_compact(sh, full, None, P, 0.5, rag, None, ws, s, check=False) == ac.ERR_INVALID_ARG
    # a cache packed behind others in shared buffers: first_row counts against the capacity, and is not negative
    rows = ac.aircache_total_rows(sh, 0.5)
    assert ac.aircache_compact(sh, full, P, P, 0.5, ac.Ragged(P, P, P, P, rows + 6, 7), None, ws, s,
                               check=False) == ac.ERR_CAPACITY
    assert ac.aircache_compact(sh, full, P, P, 0.5, ac.Ragged(P, P, P, P, rows, -1), None, ws, s,
                               check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_budget(sh, P, 0.5, 0, P, None, None, ac.Ragged(P, P, P, P, rows, -1), ws, s,
                              check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_decode_attn(sh, ac.Ragged(P, P, P, P, 10, 10), P, P, ws, s, check=False) == ac.ERR_CAPACITY
    # decode
    assert ac.aircache_decode_attn(sh, rag, None, P, ws, s, check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_decode_attn(sh, rag, P, P + 4, ws, s, check=False) == ac.ERR_ALIGNMENT
    assert ac.aircache_decode_attn(sh, ac.Ragged(None, P, P, P, 10), P, P, ws, s, check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_decode_attn(sh, ac.Ragged(P, P, P, P, 0), P, P, ws, s, check=False) == ac.ERR_CAPACITY
    # fused step: slack is 0, so the append overflows; NULL token
    assert ac.aircache_decode_step(sh, rag, P, P, P, 0, P, ws, s, check=False) == ac.ERR_CAPACITY
    assert ac.aircache_decode_step(sh, rag, P, None, P, 0, P, ws, s, check=False) == ac.ERR_INVALID_ARG
    # append: slack is 0, so any append overflows
    assert ac.aircache_append(sh, rag, P, P, 0, s, check=False) == ac.ERR_CAPACITY
    # status helpers
    assert ac.aircache_reset_status(None, s, check=False) == ac.ERR_INVALID_ARG
    assert ac.aircache_check_status(Ws(P, 8), s, check=False) == ac.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(ac.AirCacheError) as e:
        ac.aircache_decode_attn(sh, rag, None, P, ws, s)
    assert e.value.code == ac.ERR_INVALID_ARG


def test_binding_has_no_fallback(monkeypatch, tmp_path):
    """With the shared library missing the binding raises instead of computing anything some other way."""
    monkeypatch.setattr(ac, "_lib", None)
    monkeypatch.setattr(ac, "LIB", str(tmp_path / "libaircache.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        ac.aircache_version()

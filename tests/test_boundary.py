"""Host-side checks of the C-ABI: the library loads, exports every function include/sjd.h declares,
and rejects bad arguments before touching a device.  No GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2410_01699_b200 import binding as B
from paper_2410_01699_b200.inputs import WORKLOADS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sjd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sjd_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    names = _declared_functions()
    assert "sjd_init" in names and "sjd_step" in names and "sjd_verify" in names and len(names) >= 12
    lib = B.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == sorted(n for n in names)


def test_struct_sizes_match_the_header_layout():
    assert C.sizeof(B.sjd_model_cfg) == 15 * 4
    assert C.sizeof(B.sjd_weights) == 14 * 8
    assert C.sizeof(B.sjd_sample_cfg) == 48
    assert B.sjd_sample_cfg.guidance.offset == 36 and B.sjd_sample_cfg.schedule.offset == 40
    assert B.sjd_sample_cfg.seed.offset == 8 and B.sjd_sample_cfg.window.offset == 16
    assert C.sizeof(B.sjd_step_out) == 8 * 8


def test_strerror_and_status_codes():
    lib = B.lib()
    seen = set()
    for code in (0, -1, -2, -3, -4, -5, -6):
        msg = lib.sjd_strerror(code).decode()
        assert msg and msg not in seen
        seen.add(msg)
    assert "unknown" in lib.sjd_strerror(-99).decode()


def test_workspace_size_query():
    wl = WORKLOADS["7b"]
    cfg = B.make_model_cfg(wl, max_batch=1, max_seq=2432, max_window=32)
    nbytes = B.sjd_workspace_bytes(cfg)
    kv = 32 * 2 * 32 * 128 * 2432 * 2
    logits = 2 * 32 * 65536 * 2
    assert kv + logits < nbytes < kv + logits + (256 << 20)
    # paged cache: the pool (plus its spare page) replaces max_batch x max_seq rows
    paged = B.make_model_cfg(wl, max_batch=8, max_seq=2432, max_window=32, kv_pages=40)
    pool = 41 * 32 * 2 * 32 * 64 * 128 * 2
    rest = B.sjd_workspace_bytes(B.make_model_cfg(wl, 8, 2432, 32)) - 8 * kv
    assert pool + rest <= B.sjd_workspace_bytes(paged) < pool + rest + (1 << 20)
    for field, bad in (("n_layers", 0), ("head_dim", 63), ("n_kv_heads", 5), ("max_window", 0), ("dtype", 7),
                       ("kv_pages", -1)):
        c = B.make_model_cfg(wl, 1, 2432, 32)
        setattr(c, field, bad)
        assert B.sjd_workspace_bytes(c) == 0, field


def test_calls_reject_bad_arguments_without_a_device():
    lib = B.lib()
    s = B.make_sample_cfg(top_k=10, window=4)
    out = B.sjd_step_out()
    one = C.c_void_p(256)  # never dereferenced: validation fails first
    assert lib.sjd_verify(0, 4, 16, 0, one, one, one, None, None, C.byref(s), 0, C.byref(out), one, 1 << 20, None) == B.SJD_ERR_BAD_ARG
    assert lib.sjd_verify(1, 4, 16, 9, one, one, one, None, None, C.byref(s), 0, C.byref(out), one, 1 << 20, None) == B.SJD_ERR_UNSUPPORTED
    assert lib.sjd_verify(1, 65, 16, 0, one, one, one, None, None, C.byref(s), 0, C.byref(out), one, 1 << 20, None) == B.SJD_ERR_CAPACITY
    assert lib.sjd_verify(1, 4, 16, 0, one, one, one, None, None, C.byref(s), 0, C.byref(out), one, 8, None) == B.SJD_ERR_CAPACITY
    assert lib.sjd_verify(1, 4, 16, 0, None, one, one, None, None, C.byref(s), 0, C.byref(out), one, 1 << 20, None) == B.SJD_ERR_BAD_ARG
    ctx = C.c_void_p()
    cfg = B.make_model_cfg(WORKLOADS["tiny"], 1, 64, 8)
    assert lib.sjd_init(C.byref(ctx), C.byref(cfg), None, one, 1 << 30) == B.SJD_ERR_BAD_ARG
    assert lib.sjd_step(None, None, None) == B.SJD_ERR_BAD_ARG
    assert lib.sjd_prefill(None, 1, one, 4, C.byref(s), None) == B.SJD_ERR_BAD_ARG
    assert lib.sjd_last_device_status(None) == B.SJD_ERR_BAD_ARG
    lib.sjd_destroy(None)
    assert B.sjd_verify_workspace_bytes(0, 4) == 0 and B.sjd_verify_workspace_bytes(32, 32) >= 32 * 32 * 64


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libsjd.so")
    with pytest.raises(RuntimeError, match="not built"):
        B.lib()

"""The C-ABI library builds, loads and exports every function include/dba.h declares (no GPU needed)."""
import ctypes as C
import os
import re

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "dba.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dba_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_function():
    from paper_1804_06609_b200 import binding, build
    build.build()
    L = binding.lib()
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(L, n), f"{n} is declared in dba.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_host_side_argument_checks_need_no_gpu():
    from paper_1804_06609_b200 import binding
    L = binding.lib()
    so = np.array([0, 2], np.int32); po = np.array([0, 2, 3], np.int32); tk = np.array([5, 6, 7], np.int32)
    mk = lambda **kw: binding.Config(**{**dict(B=1, k=5, V=1000, max_steps=20, pad_id=0, bos_id=1, eos_id=2,
                                               logit_dtype=0, flags=0, sent_phrase_off=so.ctypes.data,
                                               phrase_tok_off=po.ctypes.data, tok=tk.ctypes.data), **kw})
    n = C.c_size_t()
    assert L.dba_workspace_bytes(C.byref(mk()), C.byref(n)) == 0 and n.value > 0 and n.value % 256 == 0
    small = n.value
    assert L.dba_workspace_bytes(C.byref(mk(flags=4)), C.byref(n)) == 0 and n.value >= small + 5 * 1000 * 4
    assert L.dba_workspace_bytes(C.byref(mk(k=65)), C.byref(n)) == 2
    assert L.dba_workspace_bytes(C.byref(mk(V=7)), C.byref(n)) == 1          # constraint token 7 >= V
    assert L.dba_workspace_bytes(C.byref(mk(logit_dtype=3)), C.byref(n)) == 1
    assert L.dba_workspace_bytes(C.byref(mk(flags=64)), C.byref(n)) == 1
    assert L.dba_workspace_bytes(None, C.byref(n)) == 1
    assert L.dba_workspace_bytes(C.byref(mk(prune_threshold=float("nan"))), C.byref(n)) == 1
    assert L.dba_workspace_bytes(C.byref(mk(prune_threshold=-1.0)), C.byref(n)) == 0     # <= 0: no pruning
    assert L.dba_workspace_bytes(C.byref(mk(prune_threshold=20.0)), C.byref(n)) == 0
    assert L.dba_counters(None, (C.c_uint32 * 4)()) == 1
    assert L.dba_status_string(0) == b"ok" and L.dba_status_string(5) == b"device-side wait timed out"
    assert L.dba_step(None, None, 0, None, None) == 1
    assert L.dba_launch_count(None) == 0
    L.dba_destroy(None)
    assert L.dba_row_scan_scratch_bytes(4, 100, 67, 0, C.byref(n)) == 2
    assert L.dba_row_scan_scratch_bytes(4, 100, 8, 0, C.byref(n)) == 0 and n.value > 0


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_1804_06609_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "missing.so"))
    try:
        binding.lib()
    except ImportError as e:
        assert "no CPU fallback" in str(e)
    else:
        raise AssertionError("a missing library must raise")

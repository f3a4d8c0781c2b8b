"""The C-ABI library builds, loads and exports every symbol include/cfgzip.h declares (no GPU needed)."""
import ctypes
import os
import re

import numpy as np

import synth
from paper_2605_29986_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "cfgzip.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cfgzip_[a-z_]+)\s*\(", text)))


def test_header_and_binding_list_the_same_calls():
    assert _declared() == sorted(binding.EXPORTED_SYMBOLS)


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(binding.load_library()._name)
    for name in _declared():
        assert hasattr(lib, name), name


def test_status_strings():
    assert binding.cfgzip_status_string(0) == "CFGZIP_OK"
    for code in range(-6, 0):
        assert binding.cfgzip_status_string(code).startswith("CFGZIP_E_")
    assert "unknown" in binding.cfgzip_status_string(-99)


def test_check_partition_on_host():
    p = synth.zipf_partition(5000, 100, 1.1, seed=1)
    assert binding.cfgzip_check_partition(p.c, p.V, p.r, p.K) == binding.OK
    bad = p.c.copy(); bad[17] = 100
    assert binding.cfgzip_check_partition(bad, p.V, p.r, p.K) == binding.E_PARTITION
    bad = p.c.copy(); bad[17] = -1
    assert binding.cfgzip_check_partition(bad, p.V, p.r, p.K) == binding.E_PARTITION
    r = p.r.copy(); r[3] = p.r[4]  # representative of another class
    assert binding.cfgzip_check_partition(p.c, p.V, r, p.K) == binding.E_PARTITION
    r = p.r.copy(); r[0] = p.V
    assert binding.cfgzip_check_partition(p.c, p.V, r, p.K) == binding.E_PARTITION
    empty = p.c.copy(); empty[empty == 7] = 8  # class 7 has no member left
    assert binding.cfgzip_check_partition(empty, p.V, p.r, p.K) == binding.E_PARTITION
    assert binding.cfgzip_check_partition(None, p.V, p.r, p.K) == binding.E_ARG
    assert binding.cfgzip_check_partition(p.c, 0, p.r, p.K) == binding.E_ARG
    assert binding.cfgzip_check_partition(p.c, 50, p.r, 100) == binding.E_ARG


def test_class_lists_on_host():
    p = synth.zipf_partition(3000, 77, 1.1, seed=2)
    off = np.empty(p.K + 1, dtype=np.int32)
    tok = np.empty(p.V, dtype=np.int32)
    assert binding.cfgzip_build_class_lists(p.c, p.V, p.K, off, tok) == binding.OK
    assert off[0] == 0 and off[-1] == p.V
    assert np.array_equal(np.diff(off), np.bincount(p.c, minlength=p.K))
    for k in range(p.K):
        seg = tok[off[k]:off[k + 1]]
        assert np.all(p.c[seg] == k) and np.all(np.diff(seg) > 0)
    assert binding.cfgzip_build_class_lists(p.c, p.V, 5, off, tok) == binding.E_PARTITION


def test_null_context_is_rejected_without_touching_a_gpu():
    assert binding.load_library().cfgzip_destroy(None) == binding.E_ARG
    assert binding.load_library().cfgzip_set_tuning(None, b"pdl", 1) == binding.E_ARG
    assert binding.load_library().cfgzip_map_tokens(None, 0, None, None, None, 1, None) == binding.E_ARG

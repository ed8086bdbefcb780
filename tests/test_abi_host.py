"""Host-side checks that need no GPU: the library loads, exports every declared symbol,
rejects bad arguments before touching CUDA, and the footprint report equals the oracle's."""
import ctypes
import os
import re

import pytest
import torch

import oracle
import paper_1905_04035_b200 as dst
from paper_1905_04035_b200 import binding
from paper_1905_04035_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def test_every_declared_symbol_is_exported():
    text = ""
    inc = os.path.join(ROOT, "include")
    for name in sorted(os.listdir(inc)):
        if name.endswith(".h"):
            text += open(os.path.join(inc, name)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(dst_[a-z_0-9]+)\s*\(", text))
    assert {"dst_densify", "dst_densify_concat", "dst_bytes_report", "dst_workspace_bytes"} <= declared
    lib = ctypes.CDLL(dst.library_path())
    for sym in declared:
        assert hasattr(lib, sym), "library does not export %s" % sym
    assert declared == set(binding.SYMBOLS), "binding and header disagree"


def test_version_and_status_strings():
    assert dst.dst_version() >= 100
    for code, name in dst.DST_STATUS.items():
        assert dst.dst_status_string(code) and "unknown" not in dst.dst_status_string(code), name
    assert "unknown" in dst.dst_status_string(99)


def test_workspace_size_grows_with_the_problem_and_rejects_bad_shapes():
    a = dst.dst_workspace_bytes(25600, 1, 1024, 33708)
    b = dst.dst_workspace_bytes(655360, 64, 1024, 33708)
    assert 0 < a < b
    assert dst.dst_workspace_bytes(-1, 1, 8, 8) == 0
    assert dst.dst_workspace_bytes(1 << 31, 1, 8, 8) == 0
    assert dst.dst_workspace_bytes(8, 1, 8, (1 << 30) + 1) == 0


def _call(slices, R, d, vocab, out, ws, ws_bytes, opts=(1, 0, 0, 0)):
    lib = dst.load_library()
    o = binding._Opts(*opts)
    arr = (binding._Slice * max(1, len(slices)))()
    for i, (a, b, n) in enumerate(slices):
        arr[i].indices, arr[i].values, arr[i].n_rows = a, b, n
    return lib.dst_densify_concat(arr, R, d, vocab, None, out, None, ctypes.byref(o), ws, ws_bytes, None, None, None)


def test_bad_arguments_are_rejected_on_the_host():
    # none of these reach a CUDA call: pointers are fake but never dereferenced
    fake = 0x1000
    need = dst.dst_workspace_bytes(100, 1, 64, 1000)
    assert _call([(fake, fake, 100)], 1, 64, 1000, fake, fake, need - 1) == 3      # workspace too small
    assert _call([(fake, fake, 100)], 1, 64, 1000, None, fake, need) == 1          # no output
    assert _call([(fake, fake, 100)], 1, 64, 1000, fake, None, need) == 1          # no workspace
    assert _call([(fake, fake, 100)], 1, 64, 1000, fake, fake + 8, need) == 1      # misaligned workspace
    assert _call([(fake, fake, -1)], 1, 64, 1000, fake, fake, need) == 1           # negative rows
    assert _call([(None, fake, 5)], 1, 64, 1000, fake, fake, need) == 1            # null indices
    assert _call([(fake, fake, 5)], -1, 64, 1000, fake, fake, need) == 1           # negative R
    assert _call([(fake, fake, 5)], 1, -64, 1000, fake, fake, need) == 1
    assert _call([(fake, fake, 5)], 1, 64, 1000, fake, fake, need, opts=(7, 0, 0, 0)) == 2   # unknown index type
    assert _call([(fake, fake, 5)], 1, 64, 1000, fake, fake, need, opts=(1, 0, 0, 1)) == 2   # unknown flag
    assert _call([(fake, fake, 1 << 30)], 1, 64, 1000, fake, fake, need) == 2      # too many rows
    assert _call([(fake, fake, 5)], 1, 64, 0, None, None, 0) == 0                  # vocab == 0: nothing to do
    assert _call([(fake, fake, 5)], 1, 0, 10, None, None, 0) == 0                  # d == 0: nothing to do


def test_bytes_report_equals_the_oracle():
    cases = (([10000] * 64, 1024, 33708, "i64", "f32", "f32"), ([10240] * 64, 1024, 33708, "i64", "f32", "f32"),
             ([1048576], 1024, 65536, "i32", "bf16", "bf16"), ([4096, 4096], 512, 33708, "i64", "f32", "bf16"),
             ([], 8, 10, "i64", "f32", "f32"), ([0, 0], 8, 0, "i32", "bf16", "f32"))
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16, "i32": torch.int32, "i64": torch.int64}
    for ns, d, vocab, it, vt, ot in cases:
        got = dst.dst_bytes_report(ns, d, vocab, tdt[it], tdt[vt], tdt[ot])
        want = oracle.bytes_report(ns, d, vocab, index_dtype=it, value_dtype=vt, out_dtype=ot)
        for k, v in want.items():
            assert got[k] == v or abs(got[k] - v) <= 1e-12 * abs(v), (k, got[k], v)


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", os.path.join(ROOT, "no_such_library.so"))
    with pytest.raises(ImportError):
        dst.dst_version()

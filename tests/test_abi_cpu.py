"""The C-ABI library on a machine without a GPU: it loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything could be launched."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2608_15533_b200 as dl
from paper_2608_15533_b200 import binding, build

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return dl.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = (ROOT / "include" / "deltalog.h").read_text()
    declared = set(re.findall(r"\b(deltalog_[a-z_]+)\s*\(", header))
    assert set(binding.EXPORTS) <= declared and len(declared) >= 7
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_status_strings(lib):
    assert dl.version() >= 100
    assert dl.status_string(0) == "ok"
    texts = {dl.status_string(c) for c in range(0, 7)}
    assert len(texts) == 7 and "unknown status code" in texts


def _desc(**kw):
    base = dict(op=dl.GDN, num_slots=4, H=2, d_k=64, d_v=64, cap=8, io_dtype=dl.BF16)
    base.update(kw)
    return dl.Desc(**base).c_struct()


def _state(null=None):
    # fake, 16-byte aligned, never dereferenced: every call below is rejected on the host
    vals = {n: 0x1000 * (i + 1) for i, n in enumerate(("S_base", "K_log", "U_log", "decay_log", "log_len", "status"))}
    if null:
        vals[null] = None
    return binding._State(**vals)


def _decode(lib, d, s, q=0x10000, k=0x20000, v=0x30000, g=0x40000, beta=0x50000, bonus=None, B=1, out=0x60000):
    return lib.deltalog_decode_step(ctypes.byref(d), ctypes.byref(s), q, k, v, g, beta, bonus, None, B, out, None)


def test_host_side_rejections_launch_nothing(lib):
    before = dl.launch_count()
    s = _state()
    assert _decode(lib, _desc(op=7), s) == binding.ERR_INVALID_ARG
    assert _decode(lib, _desc(d_k=96, d_v=96), s) == binding.ERR_UNSUPPORTED_SHAPE
    assert _decode(lib, _desc(d_k=64, d_v=96), s) == binding.ERR_UNSUPPORTED_SHAPE
    assert _decode(lib, _desc(d_k=256, d_v=128), s) == binding.ERR_UNSUPPORTED_SHAPE
    assert _decode(lib, _desc(cap=0), s) == binding.ERR_CAP_RANGE
    assert _decode(lib, _desc(cap=65), s) == binding.ERR_CAP_RANGE
    # a 16-bit U log for the delta rule needs 16-bit I/O; where b = v the U log has the I/O dtype
    assert _decode(lib, _desc(io_dtype=dl.F32, klog_dtype=dl.F32, ulog_dtype=dl.BF16), s) == binding.ERR_UNSUPPORTED_SHAPE
    assert _decode(lib, _desc(op=dl.RWKV6, ulog_dtype=dl.F32), s, bonus=0x70000) == binding.ERR_UNSUPPORTED_SHAPE
    assert _decode(lib, _desc(klog_dtype=dl.F32), s) == binding.ERR_UNSUPPORTED_SHAPE
    assert _decode(lib, _desc(num_slots=0), s) == binding.ERR_INVALID_ARG
    assert _decode(lib, _desc(), _state(null="S_base")) == binding.ERR_INVALID_ARG
    assert _decode(lib, _desc(), _state(null="log_len")) == binding.ERR_INVALID_ARG
    assert _decode(lib, _desc(), s, q=None) == binding.ERR_INVALID_ARG
    assert _decode(lib, _desc(), s, q=0x10004) == binding.ERR_INVALID_ARG                 # misaligned
    assert _decode(lib, _desc(), s, beta=None) == binding.ERR_INVALID_ARG                 # delta rule needs beta
    assert _decode(lib, _desc(op=dl.RWKV6), s, bonus=None) == binding.ERR_INVALID_ARG     # RWKV6 needs the bonus
    assert _decode(lib, _desc(), s, B=-1) == binding.ERR_INVALID_ARG
    assert _decode(lib, _desc(), s, B=0) == binding.OK                                    # empty batch: no launch
    d = _desc()
    assert lib.deltalog_merge(ctypes.byref(d), ctypes.byref(s), None, 5, 0, None) == binding.ERR_INVALID_ARG
    assert lib.deltalog_merge(ctypes.byref(d), ctypes.byref(s), None, -1, 0, None) == binding.ERR_INVALID_ARG
    assert lib.deltalog_merge(ctypes.byref(d), ctypes.byref(s), None, 0, 0, None) == binding.OK
    assert lib.deltalog_eager_step(ctypes.byref(d), None, 1, 1, 1, 1, 1, None, None, 1, 1, None, None) == \
        binding.ERR_INVALID_ARG
    assert lib.deltalog_decode_step(None, ctypes.byref(s), 1, 1, 1, 1, 1, None, None, 1, 1, None) == \
        binding.ERR_INVALID_ARG
    assert dl.launch_count() == before


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", tmp_path / "libdeltalog.so")
    with pytest.raises(ImportError, match="no fallback"):
        binding.load_library()


def test_product_package_does_not_touch_the_oracle():
    for path in (ROOT / "paper_2608_15533_b200").rglob("*"):
        if path.suffix in {".py", ".cu", ".cuh", ".h"}:
            assert "oracle" not in path.read_text(), path
    for path in (ROOT / "oracle").rglob("*.py"):
        text = path.read_text()
        assert "paper_2608_15533_b200" not in text and "libdeltalog" not in text, path

"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "mxfp4.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mxfp4_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    from paper_2502_20853_b200 import build
    path = build.build()
    assert os.path.exists(path)
    import paper_2502_20853_b200 as mx
    L = mx.lib()
    syms = _declared_symbols()
    assert len(syms) >= 12
    for s in syms:
        assert hasattr(L, s), "library does not export %s" % s
    assert sorted(mx.EXPORTS) == [s for s in syms if s in mx.EXPORTS]
    assert set(mx.EXPORTS) <= set(syms)


def test_scale_layout_host_functions():
    import paper_2502_20853_b200 as mx
    # rows pad to 128, 32-column blocks pad to 4
    assert mx.scale_bytes(1024, 192) == 8 * 2 * 512
    assert mx.scale_bytes(1, 32) == 512
    assert mx.scale_bytes(129, 32 * 5) == 2 * 2 * 512
    cols = 192
    seen = set()
    for r in range(256):
        for b in range(6):
            o = mx.scale_offset(r, b, cols)
            assert 0 <= o < mx.scale_bytes(256, cols)
            seen.add(o)
    assert len(seen) == 256 * 6  # injective
    # inside one 128x4 tile: 16 bytes per (row % 32), 4 bytes per 32-row quarter, 1 per block
    assert mx.scale_offset(0, 1, cols) == 1 and mx.scale_offset(1, 0, cols) == 16
    assert mx.scale_offset(32, 0, cols) == 4 and mx.scale_offset(0, 4, cols) == 512
    assert mx.scale_offset(128, 0, cols) == 1024


def test_missing_library_fails_loudly(monkeypatch):
    import paper_2502_20853_b200.binding as b
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", "/nonexistent/libmxfp4.so")
    with pytest.raises(RuntimeError):
        b.lib()

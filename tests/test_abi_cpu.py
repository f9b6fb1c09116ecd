"""The C-ABI library builds, loads without a GPU, and exports every symbol include/fastar.h declares.
No compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2602_01801_b200 import build, fastar
    build.build_library()
    return fastar.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "fastar.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fastar_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    from paper_2602_01801_b200 import fastar
    names = _declared()
    assert {"fastar_tempcache_update", "fastar_annsa_attention", "fastar_annca_attention", "fastar_cache_create",
            "fastar_cache_reset"} <= set(names)
    raw = ctypes.CDLL(fastar.library_path())
    for n in names:
        assert hasattr(raw, n), n
        assert n in fastar.SIGNATURES, f"{n} has no Python binding"
    assert set(fastar.SIGNATURES) == set(names)


def test_host_only_calls(lib):
    from paper_2602_01801_b200 import fastar
    assert lib.fastar_status_string(0) == b"ok"
    assert b"capacity" in lib.fastar_status_string(fastar.ERR_CAPACITY)
    d = fastar.CacheDesc(12, 128, 32768, 128, 0, 4, 8, 4680, 512, 4, fastar.BF16, 0)
    nbytes = lib.fastar_cache_workspace_bytes(ctypes.byref(d))
    pools = 2 * 12 * 32768 * 128 * 2
    assert pools < nbytes < pools * 1.6 and nbytes % 1024 == 0
    for bad in (dict(head_dim=96), dict(capacity=1000), dict(page_tokens=32), dict(lsh_bits=9), dict(max_tokens=0)):
        kw = dict(num_heads=12, head_dim=128, capacity=32768, page_tokens=128, n_sink=0, lsh_tables=4, lsh_bits=8,
                  max_tokens=4680, max_prompt_tokens=512, max_frames=4, dtype=0, device=0)
        kw.update(bad)
        assert lib.fastar_cache_workspace_bytes(ctypes.byref(fastar.CacheDesc(**kw))) == 0
    assert lib.fastar_cache_destroy(None) == fastar.ERR_INVALID_ARG
    assert lib.fastar_launch_count(None) == 0


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2602_01801_b200 import fastar
    monkeypatch.setattr(fastar, "_lib", None)
    monkeypatch.setattr(fastar, "_LIB_PATH", "/nonexistent/libfastar.so")
    with pytest.raises(RuntimeError):
        fastar.load_library()

"""The C-ABI library loads and exports every symbol include/nm.h declares (no compute, no GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2507_17301_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "nm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nm_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_three_calls():
    names = _declared()
    for must in ("nm_prune", "nm_conv2d", "nm_autotune"):
        assert must in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared():
        assert hasattr(lib, name), f"{name} is declared in nm.h but not exported"


def test_binding_names_match_header(lib_path):
    from paper_2507_17301_b200 import nm
    assert sorted(nm.EXPORTS) == _declared()
    for name in nm.EXPORTS:
        assert hasattr(nm, name) or hasattr(nm._lib, name)


def test_plan_struct_matches_the_header(lib_path):
    """nm_plan_t is plain data that crosses the ABI: the binding's field order and size are the header's."""
    from paper_2507_17301_b200 import nm
    text = open(os.path.join(ROOT, "include", "nm.h")).read()
    body = re.search(r"typedef struct \{([^}]*)\} nm_plan_t;", text).group(1)
    fields = re.findall(r"int\s+(\w+)(?:\[(\d+)\])?;", body)
    names = [n for n, _ in fields]
    ints = sum(int(c) if c else 1 for _, c in fields)
    assert names == [n for n, _ in nm.nm_plan_t._fields_]
    assert ctypes.sizeof(nm.nm_plan_t) == 4 * ints == 64
    assert [getattr(nm.nm_plan_t, n).offset for n in names[:5]] == [0, 4, 8, 12, 16]


def test_argument_errors_without_gpu(lib_path):
    from paper_2507_17301_b200 import nm
    out = ctypes.c_void_p()
    assert nm._lib.nm_prune(None, 8, 1, 1, 8, 2, 4, 8, None, ctypes.byref(out)) == nm.NM_ERR_INVALID_ARG
    assert "NULL" in nm.nm_last_error()
    fake = ctypes.c_void_p(16)
    assert nm._lib.nm_prune(fake, 8, 1, 1, 8, 5, 4, 8, None, ctypes.byref(out)) == nm.NM_ERR_INVALID_ARG
    assert nm._lib.nm_prune(fake, 8, 1, 1, 8, 0, 4, 8, None, ctypes.byref(out)) == nm.NM_ERR_INVALID_ARG
    assert nm._lib.nm_prune(fake, 8, 3, 3, 8192, 2, 4, 8, None, ctypes.byref(out)) == nm.NM_ERR_UNSUPPORTED
    assert nm._lib.nm_prune(fake, 8, 1, 1, 8, 2, 4, 512, None, ctypes.byref(out)) == nm.NM_ERR_UNSUPPORTED
    assert nm._lib.nm_weights_dims(None, None, None, None, None, None) == nm.NM_ERR_INVALID_ARG
    assert nm._lib.nm_weights_free(None) == nm.NM_OK
    assert nm._status_string(nm.NM_ERR_TIMEOUT) == "NM_ERR_TIMEOUT"


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2507_17301_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                for needle in ("import oracle", "from oracle", "nm_oracle", "oracle/"):
                    assert needle not in text, f"{f} reaches for the CPU oracle ({needle})"


def test_plan_cache_file_round_trip(lib_path, tmp_path):
    """The plan cache is host-side text: store, look up, last line of a key wins, missing entries are reported."""
    from paper_2507_17301_b200 import nm
    path = str(tmp_path / "plans.txt")
    key = nm.nm_plan_key(256, 3, 3, 256, 2, 4, 64, (64, 14, 14, 256), 1, 1, 1, True, True)
    other = nm.nm_plan_key(256, 3, 3, 256, 2, 4, 128, (64, 14, 14, 256), 1, 1, 1, True, True)
    assert key != other and " " not in key and "t64" in key and "t128" in other
    assert nm.nm_plan_cache_lookup(path, key) is None                      # no file yet
    p = nm.nm_plan_t()
    p.variant, p.bn, p.stages, p.split, p.kblk, p.loads, p.issuers, p.ksplit = 8, 256, 2, 0, 0, 2, 4, 3
    nm.nm_plan_cache_store(path, key, p)
    assert nm.nm_plan_cache_lookup(path, other) is None                    # another layer
    got = nm.nm_plan_cache_lookup(path, key)
    assert got.as_dict() == p.as_dict()
    p.variant, p.bn, p.ksplit = 4, 128, 0
    nm.nm_plan_cache_store(path, key, p)                                   # a newer entry replaces the older one
    assert nm.nm_plan_cache_lookup(path, key).as_dict() == p.as_dict()
    assert len(open(path).read().splitlines()) == 2
    with pytest.raises(nm.NmError) as e:
        nm.nm_plan_cache_store(path, "a key with blanks", p)
    assert e.value.status == nm.NM_ERR_INVALID_ARG
    buf = ctypes.create_string_buffer(8)                                   # a key buffer that is too small
    assert nm._lib.nm_plan_key(*([1] * 18), buf, len(buf)) == nm.NM_ERR_INVALID_ARG

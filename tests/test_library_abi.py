"""Host-side checks of the C-ABI library that need no GPU: it builds for sm_100a,
loads, exports every function the header declares, and its host-only helpers work."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as entry
    entry.build()
    from paper_2507_08771_b200 import binding
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "blockffn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"BLOCKFFN_API\s+[\w\s\*]+?\b(blockffn_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 12, names
    for n in names:
        assert getattr(lib, n) is not None
    from paper_2507_08771_b200 import binding
    assert sorted(binding.EXPORTS) == names
    for n in names:                       # the binding offers each call under the same name
        assert hasattr(binding, n) or n == "blockffn_status_string"


def test_host_only_helpers(lib):
    from paper_2507_08771_b200 import binding
    s = binding.Stats(n_tokens=80, n_active=768, n_chunks=10, n_union=190)
    assert binding.blockffn_tls(s, 64) == pytest.approx(1 - 768 / (80 * 64))
    assert binding.blockffn_cls(s, 64) == pytest.approx(1 - 190 / (10 * 64))
    assert binding.status_string(binding.OK) == "ok"
    assert "argument" in binding.status_string(binding.ERR_INVALID_ARG)


def test_create_rejects_bad_configs_before_touching_the_device(lib):
    from paper_2507_08771_b200 import binding
    h = ctypes.c_void_p()
    bad = [
        (binding.Config(0, 16, 64, 4, 1e-6, 0, 0), binding.ERR_INVALID_ARG),
        (binding.Config(250, 16, 64, 4, 1e-6, 0, 0), binding.ERR_UNSUPPORTED),     # d % 8
        (binding.Config(256, 16, 60, 4, 1e-6, 0, 0), binding.ERR_UNSUPPORTED),     # d_e % 8
        (binding.Config(256, 2000, 64, 4, 1e-6, 0, 0), binding.ERR_UNSUPPORTED),   # E too large
        (binding.Config(256, 16, 64, 64, 1e-6, 0, 0), binding.ERR_UNSUPPORTED),    # L_max > 32
        (binding.Config(256, 16, 64, 4, -0.5, 0, 0), binding.ERR_INVALID_ARG),     # eps < 0, not the
        (binding.Config(256, 16, 64, 4, float("nan"), 0, 0), binding.ERR_INVALID_ARG),  # no-RMSNorm value
        (binding.Config(256, 16, 64, 4, 1e-6, 9, 0), binding.ERR_INVALID_ARG),
    ]
    for cfg, want in bad:
        assert lib.blockffn_create(ctypes.byref(cfg), ctypes.byref(h)) == want
        assert not h.value
    assert lib.blockffn_create(None, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert lib.blockffn_destroy(None) == binding.ERR_INVALID_ARG


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2507_08771_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.replace("the CPU checker", ""), f
